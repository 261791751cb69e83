// Top-k sparsification (Section 3.2 "Top-k sparsification", Section 5.1 "Top-k compression") fused
// with the error feedback.  Exact selection of the k entries of largest |v| over a whole d-vector,
// ties by lower index, emitted as an index-ordered (index, value) list.
//
// The order of |v| is the order of the bit pattern with the sign cleared (a 31-bit key), so the
// selection is integer work: a radix select finds the key tau of the k-th largest entry and the
// number r of entries equal to tau that still fit.  The top 12 key bits are the "bin".
//
// Pipeline with a candidate list (the library's normal path):
//   pass1      v = source (Eq. 2 / Eq. 4), written over delta.  With a usable history of threshold
//              bins it predicts a band [lo, hi] of bins for this step's threshold and, while v is
//              still in registers, (a) sets a bit in the "kept" bitmap for every entry above the
//              band, (b) appends (key, index) of every entry inside the band to a candidate list,
//              (c) counts a 256-bin histogram of the entries from 16 bins below the band upwards.
//   pick       threshold bin tb and the number of entries still to take inside it, from that
//              partial histogram; accepts it only if the k-th entry lies inside the counted range
//              and tb inside the band.
//   hist, pick only after a miss (or without history): full 4096-bin histogram of v, exact tb
//   mark       only after a miss: re-read v, rebuild bitmap and candidate list for the exact tb
//   resolve    the next 12 and the last 7 key bits from the candidate list: tau and r
//   classify   candidates with key > tau join the kept bitmap, key == tau go to the tie bitmap
//   count, scan  per-segment population counts and their exclusive prefix
//   emit       every set bit knows its output slot: write (index, value), zero the entry in delta
//              (delta = v - Q[v], Eq. 3), and on a fused server pass update x at that entry
// In the steady state v is read once and written once; the kernels marked "only after a miss"
// leave at once.  A wrong, missing or garbage history costs time, never correctness.
//
// Pipeline without a list (built-in-scratch entry point, whose scratch must stay small):
//   pass1 (full histogram) -> pick -> mark (kept + candidate bitmaps) -> refine, pick, refine, pick
//   (candidates gathered through their bitmap) -> finalize -> scan -> emit.
//
// No float atomics, no spinning; integer atomics commute and output slots come from prefix sums
// over index-ordered bitmaps, so the result does not depend on scheduling.
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

namespace {

constexpr uint32_t kBins1 = 4096;                  // key bits 30..19
constexpr uint32_t kPartBins = 256;                // bins counted by a predicting pass1
constexpr uint32_t kFloorMargin = 16;              // ... starting this many bins (one octave) below the band
constexpr uint32_t kWordsPerThread = 4;            // count / emit / refine: bitmap words per thread
constexpr uint32_t kSegWords = kThreads * kWordsPerThread;  // 1024 bitmap words per segment
constexpr uint32_t kSegElems = kSegWords * 32;     // 32768 entries
constexpr uint64_t kTile = 4096;                   // entries a CTA handles per loop trip
constexpr uint32_t kWarpBuf = 256;                 // candidate staging entries per warp
constexpr uint32_t kPredMagic = 0x70D1C7EDu;

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

// Band of bins expected to contain this step's threshold bin: the last bin, moved by the last
// change (thresholds drift while the error builds up), widened by one bin on each side.
// Returns false when there is no usable history.
__device__ __forceinline__ bool predicted_band(const TopkPred* pred, uint32_t row, uint32_t* lo, uint32_t* hi) {
  if (!pred) return false;
  const TopkPred p = pred[row];
  if (p.magic != kPredMagic || p.tb_last >= kBins1 || p.tb_prev >= kBins1) return false;
  int trend = (int)p.tb_last - (int)p.tb_prev;
  trend = max(-2, min(3, trend));
  const int c = (int)p.tb_last + trend;
  *lo = (uint32_t)max(0, min((int)p.tb_last, c) - 1);
  *hi = (uint32_t)min((int)kBins1 - 1, max((int)p.tb_last, c) + 1);
  return true;
}

__device__ __forceinline__ uint32_t band_floor(uint32_t lo) { return lo > kFloorMargin ? lo - kFloorMargin : 0u; }

// Eight neighbouring lanes each hold a 4-bit field for each of four rows; returns to lane
// (octet base + r), r < 4, the 32-bit word of row r (fields in lane order).
__device__ __forceinline__ uint32_t octet_words4(const uint32_t (&nib)[4], uint32_t lane) {
  const bool u0 = lane & 1u, u1 = lane & 2u, u2 = lane & 4u;
  // step 1: keep the rows whose bit 0 equals lane bit 0
  const uint32_t send0 = u0 ? (nib[0] | nib[2] << 4) : (nib[1] | nib[3] << 4);
  const uint32_t keep0 = u0 ? (nib[1] | nib[3] << 4) : (nib[0] | nib[2] << 4);
  const uint32_t recv0 = __shfl_xor_sync(0xffffffffu, send0, 1);
  const uint32_t a = u0 ? ((recv0 & 15u) | (keep0 & 15u) << 4) : ((keep0 & 15u) | (recv0 & 15u) << 4);
  const uint32_t b = u0 ? ((recv0 >> 4) | (keep0 >> 4) << 4) : ((keep0 >> 4) | (recv0 >> 4) << 4);
  // step 2: rows (bit0, bit0 + 2) -> keep the one whose bit 1 equals lane bit 1
  const uint32_t send1 = u1 ? a : b, keep1 = u1 ? b : a;
  const uint32_t recv1 = __shfl_xor_sync(0xffffffffu, send1, 2);
  const uint32_t q = u1 ? (recv1 | keep1 << 8) : (keep1 | recv1 << 8);
  // step 3: both halves of the octet end with the whole word
  const uint32_t recv2 = __shfl_xor_sync(0xffffffffu, q, 4);
  return u2 ? (recv2 | q << 16) : (q | recv2 << 16);
}

// Per-warp staging of candidate (key, index) pairs in shared memory.  Candidates are rare, so a
// warp collects them over many tiles and reserves room in the vector's global list with one
// atomic per flush; the order of the list is irrelevant (it is histogrammed and scattered).
struct WarpStage {
  uint2* buf;          // kWarpBuf entries of this warp (shared memory)
  uint32_t count;      // warp-uniform
  uint2* list;         // this vector's list
  uint32_t* list_count;
  uint64_t cap;

  __device__ __forceinline__ void flush(uint32_t lane) {
    if (!count) return;
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(list_count, count);
    base = __shfl_sync(0xffffffffu, base, 0);
    __syncwarp();
    for (uint32_t i = lane; i < count; i += 32)
      if ((uint64_t)base + i < cap) list[(uint64_t)base + i] = buf[i];
    __syncwarp();
    count = 0;
  }

  // sel[j] bit k flags entry k of row j, whose index is e[j] + k.  Called by all 32 lanes.
  __device__ __forceinline__ void add(const float4 (&v)[4], const uint64_t (&e)[4], const uint32_t (&sel)[4],
                                      uint32_t lane) {
    const uint32_t c = __popc(sel[0]) + __popc(sel[1]) + __popc(sel[2]) + __popc(sel[3]);
    if (__ballot_sync(0xffffffffu, c != 0) == 0) return;
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= (uint32_t)o) incl += y;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);  // <= 512
    if (count + total > kWarpBuf) flush(lane);
    if (total > kWarpBuf) {
      // a tile this dense goes straight to the list
      uint32_t base = 0;
      if (lane == 0) base = atomicAdd(list_count, total);
      base = __shfl_sync(0xffffffffu, base, 0);
      uint64_t pos = (uint64_t)base + incl - c;
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((sel[j] >> k) & 1u) {
            if (pos < cap) list[pos] = make_uint2(key_of(compc(v[j], k)), (uint32_t)(e[j] + k));
            ++pos;
          }
      return;
    }
    uint32_t pos = count + incl - c;
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((sel[j] >> k) & 1u) buf[pos++] = make_uint2(key_of(compc(v[j], k)), (uint32_t)(e[j] + k));
    count += total;
  }
};

// ================================================================ list pipeline

// ---------------------------------------------------------------- pass1
// span: entries per CTA, a multiple of kTile.  `padded` = bitmap extent in entries (whole segments).
template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1(const SrcParams src, float* v_out, uint32_t* hist, uint64_t span,
                                                         uint64_t padded, const TopkPred* pred, uint32_t* bm_gt,
                                                         uint64_t bm_stride, uint2* list, uint32_t* list_count,
                                                         uint64_t cap) {
  __shared__ uint32_t s_hist[kPartBins];
  __shared__ uint2 s_stage[(kThreads / 32) * kWarpBuf];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  uint32_t lo = 1, hi = 0;
  const bool marking = predicted_band(pred, row, &lo, &hi);
  const uint32_t floor_bin = band_floor(lo);
  // keys at the edges of the counted range and of the band; hi + 1 = 4096 gives 2^31, above every key
  const uint32_t key_floor = floor_bin << 19, key_lo = lo << 19, key_above = (hi + 1u) << 19;
  if (marking) {
    for (uint32_t b = tid; b < kPartBins; b += kThreads) s_hist[b] = 0;
    __syncthreads();
  }
  WarpStage stage;
  stage.buf = s_stage + (tid >> 5) * kWarpBuf;
  stage.count = 0;
  stage.list = list + (uint64_t)row * cap;
  stage.list_count = list_count + row;
  stage.cap = cap;
  const uint64_t d = src.d;
  const uint64_t begin = (uint64_t)blockIdx.x * span;
  // when marking, the bitmap is written for whole segments, hence the padded end
  const uint64_t end = min(begin + span, marking ? padded : d);
  float* out_row = v_out + (uint64_t)row * d;
  for (uint64_t base = begin; base < end; base += kTile) {
    float4 v[4];
    uint32_t cnt[4];
    uint64_t ee[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ee[j] = base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = ee[j] < d ? (uint32_t)min((uint64_t)4, d - ee[j]) : 0u;
    }
    src_load_tile<SRC, 4>(src, row, ee, cnt, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (cnt[j]) {
        if (src.vec && cnt[j] == 4) {
          *reinterpret_cast<float4*>(out_row + ee[j]) = v[j];
        } else {
          for (uint32_t k = 0; k < cnt[j]; ++k) out_row[ee[j] + k] = compc(v[j], k);
        }
      }
    }
    if (marking) {
      uint32_t ngt[4], ncand[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        ngt[j] = 0;
        ncand[j] = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t key = key_of(compc(v[j], k));
          if ((uint32_t)k < cnt[j] && key >= key_floor) {  // a few percent of the entries get here
            atomicAdd(&s_hist[min((key >> 19) - floor_bin, kPartBins - 1u)], 1u);
            if (key >= key_above) ngt[j] |= 1u << k;
            else if (key >= key_lo) ncand[j] |= 1u << k;
          }
        }
      }
      const uint32_t wg = octet_words4(ngt, lane);
      const uint32_t r = lane & 7u;
      if (r < 4) bm_gt[(uint64_t)row * bm_stride + (base >> 5) + r * 32u + (tid >> 3)] = wg;
      stage.add(v, ee, ncand, lane);
    }
  }
  if (marking) {
    stage.flush(lane);
    __syncthreads();
    uint32_t* h = hist + (uint64_t)row * kBins1 + floor_bin;
    for (uint32_t b = tid; b < kPartBins; b += kThreads) {
      const uint32_t c = s_hist[b];
      if (c && floor_bin + b < kBins1) atomicAdd(&h[b], c);
    }
  }
}

// ---------------------------------------------------------------- pick
// Called by all 1024 threads of a CTA.  h: 4096 counters.  Finds the bin where the count from the
// top reaches `want` and how many entries are still to take inside it: s_out[0] = bin,
// s_out[1] = remainder, s_out[2] = total count (valid after the final barrier; s_out[0..1] only if
// 1 <= want <= total).
__device__ __forceinline__ void cta_pick(const uint32_t* h, uint32_t want, uint32_t* s_warp, uint32_t* s_out) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5;
  // thread t owns bins 4*(1023 - t) .. +3, so that a forward scan over threads walks bins downwards
  const uint32_t b0 = 4u * (1023u - tid);
  const uint32_t c3 = h[b0 + 3], c2 = h[b0 + 2], c1 = h[b0 + 1], c0 = h[b0];
  const uint32_t mine = c0 + c1 + c2 + c3;
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  if (lane == 31) s_warp[wrp] = incl;
  __syncthreads();
  if (wrp == 0) {
    const uint32_t w = s_warp[lane];
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= (uint32_t)o) wi += y;
    }
    s_warp[lane] = wi - w;  // exclusive prefix of the warp totals
  }
  __syncthreads();
  const uint32_t above = s_warp[wrp] + incl - mine;  // entries in bins above this thread's four
  if (tid == 1023) s_out[2] = above + mine;
  if (want > above && want <= above + mine) {
    uint32_t cum = above, tb = b0 + 3;
    const uint32_t cs[4] = {c3, c2, c1, c0};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (want <= cum + cs[i]) { tb = b0 + 3 - i; break; }
      cum += cs[i];
    }
    s_out[0] = tb;
    s_out[1] = want - cum;
  }
  __syncthreads();
}

__device__ __forceinline__ void remember_bin(TopkPred* pred, uint32_t row, uint32_t tb, bool had) {
  if (!pred) return;
  TopkPred np;
  np.magic = kPredMagic;
  np.tb_prev = had ? pred[row].tb_last : tb;
  np.tb_last = tb;
  np.pad = 0;
  pred[row] = np;
}

// Level-1 pick, one CTA per vector.  full = 0: judge the partial histogram of a predicting pass1.
// full = 1: runs after k_topk_hist; does something only for vectors that missed.
__global__ void __launch_bounds__(1024) k_topk_pick1(uint32_t* hist, TopkState* state, uint32_t k, TopkPred* pred,
                                                     uint32_t* list_count, int full) {
  __shared__ uint32_t s_warp[32], s_out[3];
  const uint32_t tid = threadIdx.x, row = blockIdx.x;
  uint32_t* h = hist + (uint64_t)row * kBins1;
  TopkState* st = state + row;
  if (full && !st->need_full) return;
  uint32_t lo = 1, hi = 0;
  const bool had = predicted_band(pred, row, &lo, &hi);
  if (!full && !had) {  // nothing was counted
    if (tid == 0) { st->need_full = 1; st->need_mark = 1; if (list_count) list_count[row] = 0; }
    return;
  }
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; s_out[2] = 0; }
  __syncthreads();
  cta_pick(h, k, s_warp, s_out);
  for (uint32_t b = tid; b < kBins1; b += 1024) h[b] = 0;
  if (tid != 0) return;
  const uint32_t tb = s_out[0], rem = s_out[1], total = s_out[2];
  if (full) {
    st->tb1 = tb;
    st->k_rem = rem;
    st->need_mark = 1;
    remember_bin(pred, row, tb, had);
    return;
  }
  // the partial histogram is trustworthy if the k-th entry lies inside the counted range, below
  // its clamped top bin, and the bitmap and list were built for a band that contains its bin
  const uint32_t floor_bin = band_floor(lo);
  const bool hit = total >= k && tb < floor_bin + kPartBins - 1u && tb >= lo && tb <= hi;
  if (hit) {
    st->tb1 = tb;
    st->k_rem = rem;
    st->need_full = 0;
    st->need_mark = 0;
    remember_bin(pred, row, tb, true);
  } else {
    st->need_full = 1;
    st->need_mark = 1;
    if (list_count) list_count[row] = 0;  // mark will list the candidates afresh
  }
}

// ---------------------------------------------------------------- full histogram (after a miss)
__global__ void __launch_bounds__(kThreads) k_topk_hist(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                        uint32_t* hist) {
  __shared__ uint32_t s_hist[kBins1];
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  if (!state[row].need_full) return;
  for (uint32_t b = tid; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  const float* vrow = v_in + (uint64_t)row * d;
  const uint64_t ntile = (d + kTile - 1) / kTile;
  for (uint64_t tile = blockIdx.x; tile < ntile; tile += gridDim.x) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = tile * kTile + (uint64_t)(j * kThreads + tid) * 4u;
      if (e >= d) continue;
      const uint32_t cnt = (uint32_t)min((uint64_t)4, d - e);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (vec && cnt == 4) {
        v = *reinterpret_cast<const float4*>(vrow + e);
      } else {
        for (uint32_t k = 0; k < cnt; ++k) comp(v, k) = vrow[e + k];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((uint32_t)k < cnt) atomicAdd(&s_hist[key_of(compc(v, k)) >> 19], 1u);
    }
  }
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < kBins1; b += kThreads) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
}

// ---------------------------------------------------------------- mark (after a miss)
// Bitmap of the entries above the exact threshold bin and the list of those inside it.  One tile
// per loop trip over a small grid; every bitmap word up to the padded end is written.
__global__ void __launch_bounds__(kThreads) k_topk_mark(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                        uint32_t* bm_gt, uint64_t bm_stride, uint64_t padded, uint2* list,
                                                        uint32_t* list_count, uint64_t cap) {
  __shared__ uint2 s_stage[(kThreads / 32) * kWarpBuf];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  if (!state[row].need_mark) return;
  const uint32_t tb = state[row].tb1;
  const float* vrow = v_in + (uint64_t)row * d;
  WarpStage stage;
  stage.buf = s_stage + (tid >> 5) * kWarpBuf;
  stage.count = 0;
  stage.list = list + (uint64_t)row * cap;
  stage.list_count = list_count + row;
  stage.cap = cap;
  const uint64_t ntile = padded / kTile;
  for (uint64_t tile = blockIdx.x; tile < ntile; tile += gridDim.x) {
    float4 v[4];
    uint32_t cnt[4];
    uint64_t ee[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ee[j] = tile * kTile + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = ee[j] < d ? (uint32_t)min((uint64_t)4, d - ee[j]) : 0u;
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cnt[j]) {
        if (vec && cnt[j] == 4) {
          v[j] = *reinterpret_cast<const float4*>(vrow + ee[j]);
        } else {
          for (uint32_t k = 0; k < cnt[j]; ++k) comp(v[j], k) = vrow[ee[j] + k];
        }
      }
    }
    uint32_t ngt[4], ncand[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ngt[j] = 0;
      ncand[j] = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t bin = key_of(compc(v[j], k)) >> 19;
        const bool in = (uint32_t)k < cnt[j];
        ngt[j] |= (in && bin > tb ? 1u : 0u) << k;
        ncand[j] |= (in && bin == tb ? 1u : 0u) << k;
      }
    }
    const uint32_t wg = octet_words4(ngt, lane);
    const uint32_t r = lane & 7u;
    if (r < 4) bm_gt[(uint64_t)row * bm_stride + tile * (kTile / 32) + r * 32u + (tid >> 3)] = wg;
    stage.add(v, ee, ncand, lane);
  }
  stage.flush(lane);
}

// ---------------------------------------------------------------- resolve
// One CTA per vector: the second and third radix digits from the candidate list.
__global__ void __launch_bounds__(1024) k_topk_resolve(const uint2* list, const uint32_t* list_count, uint64_t cap,
                                                       TopkState* state) {
  __shared__ uint32_t s_hist[kBins1];
  __shared__ uint32_t s_warp[32], s_out[3];
  const uint32_t tid = threadIdx.x, row = blockIdx.x;
  const uint2* lrow = list + (uint64_t)row * cap;
  const uint64_t n = min((uint64_t)list_count[row], cap);
  TopkState* st = state + row;
  const uint32_t tb1 = st->tb1, want = st->k_rem;
  for (uint32_t b = tid; b < kBins1; b += 1024) s_hist[b] = 0;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; }
  __syncthreads();
  for (uint64_t i0 = 0; i0 < n; i0 += 8 * 1024) {
    uint32_t key[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint64_t i = i0 + (uint64_t)u * 1024 + tid;
      key[u] = i < n ? lrow[i].x : 0xFFFFFFFFu;  // bin 8191: never equal to tb1
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if ((key[u] >> 19) == tb1) atomicAdd(&s_hist[(key[u] >> 7) & 0xFFFu], 1u);
  }
  __syncthreads();
  cta_pick(s_hist, want, s_warp, s_out);
  const uint32_t tb2 = s_out[0], rem2 = s_out[1];
  __syncthreads();
  for (uint32_t b = tid; b < kBins1; b += 1024) s_hist[b] = 0;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; }
  __syncthreads();
  const uint32_t top24 = (tb1 << 12) | tb2;
  for (uint64_t i0 = 0; i0 < n; i0 += 8 * 1024) {
    uint32_t key[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint64_t i = i0 + (uint64_t)u * 1024 + tid;
      key[u] = i < n ? lrow[i].x : 0xFFFFFFFFu;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if ((key[u] >> 7) == top24) atomicAdd(&s_hist[key[u] & 0x7Fu], 1u);
  }
  __syncthreads();
  cta_pick(s_hist, rem2, s_warp, s_out);
  if (tid == 0) {
    st->tb2 = tb2;
    st->tau = (top24 << 7) | s_out[0];
    st->r = s_out[1];
    st->k_rem = s_out[1];
  }
}

// ---------------------------------------------------------------- classify
// Candidates above tau join the kept bitmap; candidates equal to tau are set in the tie bitmap
// (which the launcher cleared).  Candidate bits are never set in bm_gt beforehand, so the ORs
// commute with nothing else.
__global__ void __launch_bounds__(kThreads) k_topk_classify(const uint2* list, const uint32_t* list_count, uint64_t cap,
                                                            const TopkState* state, uint32_t* bm_gt, uint32_t* bm_tie,
                                                            uint64_t bm_stride) {
  const uint32_t row = blockIdx.y;
  const uint2* lrow = list + (uint64_t)row * cap;
  const uint64_t n = min((uint64_t)list_count[row], cap);
  const uint32_t tau = state[row].tau;
  uint32_t* g = bm_gt + (uint64_t)row * bm_stride;
  uint32_t* t = bm_tie + (uint64_t)row * bm_stride;
  for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (uint64_t)gridDim.x * kThreads) {
    const uint2 e = lrow[i];
    if (e.x > tau) atomicOr(&g[e.y >> 5], 1u << (e.y & 31u));
    else if (e.x == tau) atomicOr(&t[e.y >> 5], 1u << (e.y & 31u));
  }
}

// ---------------------------------------------------------------- count
// Population counts per segment (x: kept, y: ties).
__global__ void __launch_bounds__(kThreads) k_topk_count(const uint32_t* bm_gt, const uint32_t* bm_tie, uint64_t bm_stride,
                                                         uint2* seg_cnt, uint64_t nseg) {
  __shared__ uint32_t s_gt[kThreads / 32], s_tie[kThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint64_t at = (uint64_t)row * bm_stride + (uint64_t)blockIdx.x * kSegWords + tid * kWordsPerThread;
  const uint4 g4 = *reinterpret_cast<const uint4*>(bm_gt + at);
  const uint4 t4 = *reinterpret_cast<const uint4*>(bm_tie + at);
  uint32_t ng = __popc(g4.x) + __popc(g4.y) + __popc(g4.z) + __popc(g4.w);
  uint32_t nt = __popc(t4.x) + __popc(t4.y) + __popc(t4.z) + __popc(t4.w);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ng += __shfl_xor_sync(0xffffffffu, ng, o);
    nt += __shfl_xor_sync(0xffffffffu, nt, o);
  }
  if (lane == 0) { s_gt[tid >> 5] = ng; s_tie[tid >> 5] = nt; }
  __syncthreads();
  if (tid == 0) {
    uint32_t a = 0, b = 0;
    for (uint32_t i = 0; i < kThreads / 32; ++i) { a += s_gt[i]; b += s_tie[i]; }
    seg_cnt[(uint64_t)row * nseg + blockIdx.x] = make_uint2(a, b);
  }
}

// ================================================================ pipeline without a list

// pass1 with the full 4096-bin histogram and no marking.
template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1_basic(const SrcParams src, float* v_out, uint32_t* hist,
                                                               uint64_t span) {
  __shared__ uint32_t s_hist[kBins1];
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  for (uint32_t b = tid; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  const uint64_t d = src.d;
  const uint64_t begin = (uint64_t)blockIdx.x * span;
  const uint64_t end = min(begin + span, d);
  float* out_row = v_out + (uint64_t)row * d;
  for (uint64_t base = begin; base < end; base += kTile) {
    float4 v[4];
    uint32_t cnt[4];
    uint64_t ee[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ee[j] = base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = ee[j] < d ? (uint32_t)min((uint64_t)4, d - ee[j]) : 0u;
    }
    src_load_tile<SRC, 4>(src, row, ee, cnt, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (!cnt[j]) continue;
      if (src.vec && cnt[j] == 4) {
        *reinterpret_cast<float4*>(out_row + ee[j]) = v[j];
      } else {
        for (uint32_t k = 0; k < cnt[j]; ++k) out_row[ee[j] + k] = compc(v[j], k);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((uint32_t)k < cnt[j]) atomicAdd(&s_hist[key_of(compc(v[j], k)) >> 19], 1u);
    }
  }
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < kBins1; b += kThreads) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
}

// One CTA per vector, on the global histogram, which it clears for its next use.
//   level 1: bins = key >> 19            want = k
//   level 2: bins = (key >> 7) & 0xFFF   want = k_rem
//   level 3: bins = key & 0x7F           want = k_rem   -> tau and r complete
__global__ void __launch_bounds__(1024) k_topk_pick_basic(uint32_t* hist, TopkState* state, uint32_t level, uint32_t k) {
  __shared__ uint32_t s_warp[32], s_out[3];
  const uint32_t tid = threadIdx.x, row = blockIdx.x;
  uint32_t* h = hist + (uint64_t)row * kBins1;
  TopkState* st = state + row;
  const uint32_t want = level == 1 ? k : st->k_rem;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; }
  __syncthreads();
  cta_pick(h, want, s_warp, s_out);
  for (uint32_t b = tid; b < kBins1; b += 1024) h[b] = 0;
  if (tid != 0) return;
  const uint32_t tb = s_out[0], rem = s_out[1];
  st->k_rem = rem;
  if (level == 1) {
    st->tb1 = tb;
  } else if (level == 2) {
    st->tb2 = tb;
  } else {
    st->tau = (st->tb1 << 19) | (st->tb2 << 7) | tb;
    st->r = rem;
  }
}

// Two bitmaps for the exact threshold bin: bin > tb, bin == tb (the candidates).
__global__ void __launch_bounds__(kThreads) k_topk_mark_basic(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                              uint32_t* bm_gt, uint32_t* bm_eq, uint64_t bm_stride,
                                                              uint64_t padded) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint32_t tb = state[row].tb1;
  const float* vrow = v_in + (uint64_t)row * d;
  const uint64_t ntile = padded / kTile;
  for (uint64_t tile = blockIdx.x; tile < ntile; tile += gridDim.x) {
    uint32_t ngt[4], neq[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = tile * kTile + (uint64_t)(j * kThreads + tid) * 4u;
      const uint32_t cnt = e < d ? (uint32_t)min((uint64_t)4, d - e) : 0u;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cnt) {
        if (vec && cnt == 4) {
          v = *reinterpret_cast<const float4*>(vrow + e);
        } else {
          for (uint32_t k = 0; k < cnt; ++k) comp(v, k) = vrow[e + k];
        }
      }
      ngt[j] = 0;
      neq[j] = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t bin = key_of(compc(v, k)) >> 19;
        const bool in = (uint32_t)k < cnt;
        ngt[j] |= (in && bin > tb ? 1u : 0u) << k;
        neq[j] |= (in && bin == tb ? 1u : 0u) << k;
      }
    }
    const uint32_t wg = octet_words4(ngt, lane), we = octet_words4(neq, lane);
    const uint32_t r = lane & 7u;
    if (r < 4) {
      const uint64_t w = (uint64_t)row * bm_stride + tile * (kTile / 32) + r * 32u + (tid >> 3);
      bm_gt[w] = wg;
      bm_eq[w] = we;
    }
  }
}

// Histogram of the next key digit over the candidates (set bits of bm_eq), values gathered from v.
template <int LEVEL>
__global__ void __launch_bounds__(kThreads) k_topk_refine(const float* v_in, uint64_t d, const TopkState* state,
                                                          const uint32_t* bm_eq, uint64_t bm_stride, uint32_t* hist) {
  constexpr uint32_t NB = LEVEL == 2 ? 4096u : 128u;
  __shared__ uint32_t s_hist[NB];
  __shared__ uint32_t s_any;
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid * kWordsPerThread;
  const uint4 w4 = *reinterpret_cast<const uint4*>(bm_eq + (uint64_t)row * bm_stride + widx);
  const uint32_t ws[4] = {w4.x, w4.y, w4.z, w4.w};
  if (tid == 0) s_any = 0;
  __syncthreads();
  if (w4.x | w4.y | w4.z | w4.w) s_any = 1;
  __syncthreads();
  if (!s_any) return;  // uniform: no candidate in this segment
  for (uint32_t b = tid; b < NB; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  const float* vrow = v_in + (uint64_t)row * d;
  const uint32_t top24 = (state[row].tb1 << 12) | state[row].tb2;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t w = ws[i];
    while (w) {
      const uint32_t b = __ffs(w) - 1u;
      w &= w - 1u;
      const uint32_t key = key_of(vrow[(widx + i) * 32u + b]);
      if (LEVEL == 2) {
        atomicAdd(&s_hist[(key >> 7) & 0xFFFu], 1u);  // every candidate lies in the threshold bin
      } else if ((key >> 7) == top24) {
        atomicAdd(&s_hist[key & 0x7Fu], 1u);
      }
    }
  }
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < NB; b += kThreads) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
}

// bm_gt <- key > tau, bm_eq <- key == tau (candidate values gathered through the bitmap);
// population counts per segment (x: kept, y: ties).
__global__ void __launch_bounds__(kThreads) k_topk_finalize(const float* v_in, uint64_t d, const TopkState* state,
                                                            uint32_t* bm_gt, uint32_t* bm_eq, uint64_t bm_stride,
                                                            uint2* seg_cnt, uint64_t nseg) {
  __shared__ uint32_t s_gt[kThreads / 32], s_tie[kThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid * kWordsPerThread;
  const uint64_t at = (uint64_t)row * bm_stride + widx;
  const uint4 g4 = *reinterpret_cast<const uint4*>(bm_gt + at);
  const uint4 c4 = *reinterpret_cast<const uint4*>(bm_eq + at);
  uint32_t gt[4] = {g4.x, g4.y, g4.z, g4.w};
  const uint32_t cand[4] = {c4.x, c4.y, c4.z, c4.w};
  uint32_t tie[4] = {0, 0, 0, 0};
  if (c4.x | c4.y | c4.z | c4.w) {
    const float* vrow = v_in + (uint64_t)row * d;
    const uint32_t tau = state[row].tau;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t c = cand[i];
      while (c) {
        const uint32_t b = __ffs(c) - 1u;
        c &= c - 1u;
        const uint32_t key = key_of(vrow[(widx + i) * 32u + b]);
        if (key > tau) gt[i] |= 1u << b;
        else if (key == tau) tie[i] |= 1u << b;
      }
    }
    *reinterpret_cast<uint4*>(bm_gt + at) = make_uint4(gt[0], gt[1], gt[2], gt[3]);
  }
  *reinterpret_cast<uint4*>(bm_eq + at) = make_uint4(tie[0], tie[1], tie[2], tie[3]);
  uint32_t ng = __popc(gt[0]) + __popc(gt[1]) + __popc(gt[2]) + __popc(gt[3]);
  uint32_t nt = __popc(tie[0]) + __popc(tie[1]) + __popc(tie[2]) + __popc(tie[3]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ng += __shfl_xor_sync(0xffffffffu, ng, o);
    nt += __shfl_xor_sync(0xffffffffu, nt, o);
  }
  if (lane == 0) { s_gt[tid >> 5] = ng; s_tie[tid >> 5] = nt; }
  __syncthreads();
  if (tid == 0) {
    uint32_t a = 0, b = 0;
    for (uint32_t i = 0; i < kThreads / 32; ++i) { a += s_gt[i]; b += s_tie[i]; }
    seg_cnt[(uint64_t)row * nseg + blockIdx.x] = make_uint2(a, b);
  }
}

// ================================================================ shared tail

// Exclusive prefix of the per-segment counts of one vector, in place; checks that exactly k
// entries will be emitted.
__global__ void __launch_bounds__(1024) k_topk_scan(uint2* seg_cnt, uint64_t nseg, TopkState* state, uint32_t k,
                                                    uint32_t* dev_status) {
  __shared__ uint2 s_warp[32];
  __shared__ uint2 s_carry;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5, row = blockIdx.x;
  uint2* c = seg_cnt + (uint64_t)row * nseg;
  if (tid == 0) s_carry = make_uint2(0, 0);
  __syncthreads();
  for (uint64_t base = 0; base < nseg; base += 1024) {
    const uint64_t i = base + tid;
    const uint2 mine = i < nseg ? c[i] : make_uint2(0, 0);
    uint2 incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t yx = __shfl_up_sync(0xffffffffu, incl.x, o), yy = __shfl_up_sync(0xffffffffu, incl.y, o);
      if (lane >= (uint32_t)o) { incl.x += yx; incl.y += yy; }
    }
    if (lane == 31) s_warp[wrp] = incl;
    __syncthreads();
    if (wrp == 0) {
      const uint2 w = s_warp[lane];
      uint2 wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t yx = __shfl_up_sync(0xffffffffu, wi.x, o), yy = __shfl_up_sync(0xffffffffu, wi.y, o);
        if (lane >= (uint32_t)o) { wi.x += yx; wi.y += yy; }
      }
      s_warp[lane] = make_uint2(wi.x - w.x, wi.y - w.y);
    }
    __syncthreads();
    const uint2 carry = s_carry;
    const uint2 excl = make_uint2(carry.x + s_warp[wrp].x + incl.x - mine.x, carry.y + s_warp[wrp].y + incl.y - mine.y);
    if (i < nseg) c[i] = excl;
    __syncthreads();
    if (tid == 1023) s_carry = make_uint2(excl.x + mine.x, excl.y + mine.y);
    __syncthreads();
  }
  if (tid == 0) {
    const uint2 tot = s_carry;
    const uint32_t r = state[row].r;
    state[row].total_gt = tot.x;
    state[row].total_tie = tot.y;
    if (tot.x + min(tot.y, r) != k) atomicOr(dev_status, DS_DEV_TOPK_INCONSISTENT);
  }
}

__global__ void __launch_bounds__(kThreads) k_topk_emit(float* v_io, uint64_t d, const TopkState* state,
                                                        const uint32_t* bm_gt, const uint32_t* bm_eq, uint64_t bm_stride,
                                                        const uint2* seg_pre, uint64_t nseg, uint8_t* payload,
                                                        uint64_t payload_stride, uint64_t off_idx, uint64_t off_val,
                                                        uint32_t k, float* x, float gamma) {
  __shared__ uint32_t s_warp[kThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5, row = blockIdx.y;
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid * kWordsPerThread;
  const uint64_t at = (uint64_t)row * bm_stride + widx;
  const uint4 g4 = *reinterpret_cast<const uint4*>(bm_gt + at);
  const uint4 t4 = *reinterpret_cast<const uint4*>(bm_eq + at);
  const uint32_t gt[4] = {g4.x, g4.y, g4.z, g4.w};
  const uint32_t tie[4] = {t4.x, t4.y, t4.z, t4.w};
  // exclusive scan inside the segment; kept count in the low 16 bits, tie count in the high 16
  uint32_t cw[4], mine = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    cw[i] = __popc(gt[i]) | (__popc(tie[i]) << 16);
    mine += cw[i];
  }
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  if (lane == 31) s_warp[wrp] = incl;
  __syncthreads();
  uint32_t warp_pre = 0;
  for (uint32_t i = 0; i < wrp; ++i) warp_pre += s_warp[i];
  uint32_t excl = warp_pre + incl - mine;
  if (!mine) return;
  const uint2 pre = seg_pre[(uint64_t)row * nseg + blockIdx.x];
  const uint32_t r = state[row].r;
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(payload + (uint64_t)row * payload_stride + off_idx);
  float* out_val = reinterpret_cast<float*>(payload + (uint64_t)row * payload_stride + off_val);
  float* vrow = v_io + (uint64_t)row * d;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (cw[i]) {
      const uint32_t ties_before = pre.y + (excl >> 16);
      uint32_t keep = tie[i];
      const uint32_t room = r > ties_before ? r - ties_before : 0u;
      while ((uint32_t)__popc(keep) > room) keep &= ~(0x80000000u >> __clz(keep));  // drop the highest tie
      uint32_t sel = gt[i] | keep;
      uint32_t pos = pre.x + (excl & 0xFFFFu) + min(ties_before, r);
      while (sel) {
        const uint32_t b = __ffs(sel) - 1u;
        sel &= sel - 1u;
        const uint64_t j = (widx + i) * 32u + b;
        const float val = vrow[j];
        if (pos < k) {  // always true when the counts are consistent; keeps a bad count inside the payload
          out_idx[pos] = (uint32_t)j;
          out_val[pos] = val;
        }
        vrow[j] = 0.f;  // delta = v - Q[v] at a kept entry
        if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, val));
        ++pos;
      }
    }
    excl += cw[i];
  }
}

}  // namespace

void topk_plan(uint64_t d, uint32_t rows, uint64_t k, bool with_list, TopkPlan* p) {
  p->d = d;
  p->rows = rows;
  p->k = k;
  const uint64_t nw = (d + 31) / 32;
  p->nseg = (nw + kSegWords - 1) / kSegWords;
  p->bm_stride = p->nseg * kSegWords;
  p->list_cap = with_list ? d : 0;
  uint64_t pos = 0;
  p->off_hist = pos;       pos += (uint64_t)rows * kBins1 * 4;      // histogram and list counters are
  p->off_list_count = pos; pos = round16(pos + (uint64_t)rows * 4);  // cleared by one memset
  p->off_state = pos;      pos = round16(pos + (uint64_t)rows * sizeof(TopkState));
  p->off_bm_gt = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_bm_eq = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_seg = pos;        pos = round16(pos + (uint64_t)rows * p->nseg * sizeof(uint2));
  p->off_list = pos;       pos = round16(pos + (uint64_t)rows * p->list_cap * sizeof(uint2));
  p->bytes = pos;
  p->pred = nullptr;
}

cudaError_t launch_topk(int srck, const SrcParams& src, const TopkPlan& pl, void* workspace, const TopkIO& io,
                        uint32_t rows, uint64_t k, cudaStream_t st) {
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + pl.off_hist);
  uint32_t* list_count = reinterpret_cast<uint32_t*>(ws + pl.off_list_count);
  TopkState* state = reinterpret_cast<TopkState*>(ws + pl.off_state);
  uint32_t* bm_gt = reinterpret_cast<uint32_t*>(ws + pl.off_bm_gt);
  uint32_t* bm_eq = reinterpret_cast<uint32_t*>(ws + pl.off_bm_eq);  // candidates (no list) / ties
  uint2* seg = reinterpret_cast<uint2*>(ws + pl.off_seg);
  uint2* list = pl.list_cap ? reinterpret_cast<uint2*>(ws + pl.off_list) : nullptr;
  const uint64_t d = src.d, cap = pl.list_cap;
  const uint64_t padded = pl.nseg * (uint64_t)kSegElems;
  cudaError_t e = cudaMemsetAsync(hist, 0, (uint64_t)rows * kBins1 * 4 + (uint64_t)rows * 4, st);
  if (e != cudaSuccess) return e;

  // entries per CTA of pass1: enough CTAs to fill the GPU several times over
  uint64_t span = 16 * kTile;
  while (span > kTile && ((padded + span - 1) / span) * rows < 148ull * 16ull) span /= 2;
  dim3 g1((unsigned)((padded + span - 1) / span), rows, 1);
  const uint32_t k32 = (uint32_t)k;
  dim3 gs((unsigned)pl.nseg, rows, 1);
  // kernels that re-read a whole vector after a miss: a grid that fills the GPU and strides over tiles
  uint64_t stride_ctas = 148ull * 8ull / rows;
  if (stride_ctas < 1) stride_ctas = 1;
  if (stride_ctas > padded / kTile) stride_ctas = padded / kTile;
  dim3 gm((unsigned)stride_ctas, rows, 1);

  if (list && k) {
    TopkPred* pred = pl.pred;
#define DSQ_P1(S)                                                                                                 \
  k_topk_pass1<S><<<g1, kThreads, 0, st>>>(src, io.v_inout, hist, span, padded, pred, bm_gt, pl.bm_stride, list, \
                                           list_count, cap)
    switch (srck) {
      case SRC_WORKER: DSQ_P1(SRC_WORKER); break;
      case SRC_SRV_IDENTITY: DSQ_P1(SRC_SRV_IDENTITY); break;
      case SRC_SRV_SIGN1: DSQ_P1(SRC_SRV_SIGN1); break;
      case SRC_SRV_TOPK: DSQ_P1(SRC_SRV_TOPK); break;
      case SRC_SRV_QSGD: DSQ_P1(SRC_SRV_QSGD); break;
      default: return cudaErrorInvalidValue;
    }
#undef DSQ_P1
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(bm_eq, 0, (uint64_t)rows * pl.bm_stride * 4, st)) != cudaSuccess) return e;  // tie bitmap
    k_topk_pick1<<<rows, 1024, 0, st>>>(hist, state, k32, pred, list_count, 0);
    k_topk_hist<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, hist);
    k_topk_pick1<<<rows, 1024, 0, st>>>(hist, state, k32, pred, list_count, 1);
    k_topk_mark<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, bm_gt, pl.bm_stride, padded, list, list_count, cap);
    k_topk_resolve<<<rows, 1024, 0, st>>>(list, list_count, cap, state);
    dim3 gc((unsigned)(148ull * 8ull / rows ? 148ull * 8ull / rows : 1), rows, 1);
    k_topk_classify<<<gc, kThreads, 0, st>>>(list, list_count, cap, state, bm_gt, bm_eq, pl.bm_stride);
    k_topk_count<<<gs, kThreads, 0, st>>>(bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
    count_launches(8);
  } else {
#define DSQ_P1(S) k_topk_pass1_basic<S><<<g1, kThreads, 0, st>>>(src, io.v_inout, hist, span)
    switch (srck) {
      case SRC_WORKER: DSQ_P1(SRC_WORKER); break;
      case SRC_SRV_IDENTITY: DSQ_P1(SRC_SRV_IDENTITY); break;
      case SRC_SRV_SIGN1: DSQ_P1(SRC_SRV_SIGN1); break;
      case SRC_SRV_TOPK: DSQ_P1(SRC_SRV_TOPK); break;
      case SRC_SRV_QSGD: DSQ_P1(SRC_SRV_QSGD); break;
      default: return cudaErrorInvalidValue;
    }
#undef DSQ_P1
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (k == 0) return cudaSuccess;  // nothing kept: Q[v] = 0, delta = v, x unchanged
    k_topk_pick_basic<<<rows, 1024, 0, st>>>(hist, state, 1, k32);
    k_topk_mark_basic<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, bm_gt, bm_eq, pl.bm_stride, padded);
    k_topk_refine<2><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    k_topk_pick_basic<<<rows, 1024, 0, st>>>(hist, state, 2, k32);
    k_topk_refine<3><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    k_topk_pick_basic<<<rows, 1024, 0, st>>>(hist, state, 3, k32);
    k_topk_finalize<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
    count_launches(7);
  }
  k_topk_scan<<<rows, 1024, 0, st>>>(seg, pl.nseg, state, k32, io.dev_status);
  k_topk_emit<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg,
                                       reinterpret_cast<uint8_t*>(io.idx), io.payload_stride, 0,
                                       (uint64_t)(reinterpret_cast<uint8_t*>(io.val) - reinterpret_cast<uint8_t*>(io.idx)),
                                       k32, io.x, io.gamma);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace dsq
