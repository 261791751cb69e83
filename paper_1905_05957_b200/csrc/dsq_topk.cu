// Top-k sparsification (Section 3.2 "Top-k sparsification", Section 5.1 "Top-k compression") fused
// with the error feedback.  Exact selection of the k entries of largest |v| over a whole d-vector,
// ties by lower index, emitted as an index-ordered (index, value) list.
//
// The order of |v| is the order of the bit pattern with the sign cleared (a 31-bit key), so the
// selection is integer work: a radix select finds the key tau of the k-th largest entry and the
// number r of entries equal to tau that still fit.  The top 12 key bits are the "bin".
//
// Pipeline with a candidate list (the library's normal path):
//   pass1      v = source (Eq. 2 / Eq. 4), written over delta.  With the thresholds of the two
//              previous steps it predicts a band of keys [lo, hi] around this step's threshold and,
//              while v is still in registers, (a) sets a bit in the "kept" bitmap for every entry
//              above the band and counts them, (b) writes (key, index) of every entry inside the
//              band to the candidate list.  The list has one fixed region per 4096-entry tile
//              (as many slots as the tile has entries), so no reservation between CTAs is needed.
//   lhist 1    copies the tile regions into one dense list and counts the top 12 key bits on the
//              way; accepts the prediction only if the k-th entry falls inside the list
//              (kept < k <= kept + candidates)
//   hist, pick only after a miss (or without history): full 4096-bin histogram of v, exact bin tb
//   mark, compact  only after a miss: re-read v, rebuild bitmap and candidate list for the exact tb
//   lhist 2,3  the next 12, then the last 7 key bits from the candidate list: tau and r
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
constexpr uint32_t kWordsPerThread = 4;            // count / emit / refine: bitmap words per thread
constexpr uint32_t kSegWords = kThreads * kWordsPerThread;  // 1024 bitmap words per segment
constexpr uint32_t kSegElems = kSegWords * 32;     // 32768 entries
constexpr uint64_t kTile = 4096;                   // entries a CTA handles per loop trip
constexpr uint32_t kPredMagic = 0x70D1C7EDu;
constexpr uint32_t kBandHalf = 1u << 16;           // least half-width of the band in key units (0.5 % of magnitude)
constexpr uint32_t kMaxErr = 1u << 21;             // widest extrapolation error followed (band: half an octave each way)
constexpr uint32_t kFirstErr = kMaxErr;            // error assumed before any extrapolation has been checked
constexpr int kMaxTrend = 1 << 20;                 // largest step-to-step drift that is extrapolated (9 %)

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

// Keys are monotone in log-magnitude (2^23 units per octave), so a threshold that drifts by a
// steady factor moves by a steady key difference.  The band is the last threshold, extrapolated by
// the last change (the drift itself changes slowly), widened on both sides by the largest of a
// quarter of that change, 0.5 % of magnitude, and twice the recent extrapolation error (a decaying
// maximum kept beside the thresholds), so the band is wide while the error memories are still
// filling and narrows once the threshold settles.
// Candidates are the entries with lo <= key <= hi; returns false when there is no usable history.
__device__ __forceinline__ bool predicted_band(const TopkPred* pred, uint32_t row, uint32_t* lo, uint32_t* hi,
                                               uint32_t* centre = nullptr) {
  if (!pred) return false;
  const TopkPred p = pred[row];
  if (p.magic != kPredMagic || (p.tau_last | p.tau_prev) >> 31) return false;
  long long trend = (long long)p.tau_last - (long long)p.tau_prev;
  trend = max((long long)-kMaxTrend, min((long long)kMaxTrend, trend));
  const long long c = (long long)p.tau_last + trend;
  const long long err = min(p.err, kMaxErr);
  const long long half = max(max((long long)kBandHalf, 2 * err), (trend < 0 ? -trend : trend) / 4);
  if (centre) *centre = (uint32_t)max(0ll, min(0x7fffffffll, c));
  const long long l = min((long long)p.tau_last, c) - half, h = max((long long)p.tau_last, c) + half;
  *lo = (uint32_t)max(0ll, l);
  *hi = (uint32_t)min(0x7fffffffll, h);
  return true;
}

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

// Writes the candidates of one tile -- sel[j] bit k flags entry k of row j, whose key is
// keys[4 j + k] and whose index is idx0[j] + k -- into the tile's own region of the list (kTile slots, enough for every entry of
// the tile).  Slots are handed out by a shared-memory counter, one atomic per warp; the order
// inside the region is irrelevant.  Called by all 32 lanes of every warp of the CTA.
__device__ __forceinline__ void tile_append(uint2* region, uint32_t* s_count, const uint32_t (&keys)[16],
                                            const uint32_t (&idx0)[4], const uint32_t (&sel)[4], uint32_t lane) {
  const uint32_t c = __popc(sel[0]) + __popc(sel[1]) + __popc(sel[2]) + __popc(sel[3]);
  if (__ballot_sync(0xffffffffu, c != 0) == 0) return;
  uint32_t incl = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
  uint32_t base = 0;
  if (lane == 0) base = atomicAdd(s_count, total);
  base = __shfl_sync(0xffffffffu, base, 0);
  uint32_t pos = base + incl - c;
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((sel[j] >> k) & 1u) {
        if (pos < kTile) region[pos] = make_uint2(keys[4 * j + k], idx0[j] + k);
        ++pos;
      }
}

// ================================================================ list pipeline

// ---------------------------------------------------------------- pass1
// One CTA per 4096-entry tile; the grid covers the padded bitmap extent.  tile_info[tile] receives
// (candidates written, entries above the band).
template <int SRC, bool FULL>
__device__ __forceinline__ void pass1_tile(const SrcParams& src, uint32_t row, uint64_t base, float* out_row, bool marking,
                                           uint32_t key_lo, uint32_t key_hi, uint32_t* bm_row, uint2* region,
                                           uint32_t* s_count, uint32_t* s_kept) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint64_t d = src.d;
  float4 v[4];
  uint32_t cnt[4];
  if constexpr (FULL && SRC == SRC_WORKER) {
    const float4* gp = reinterpret_cast<const float4*>(src.g + (uint64_t)row * d + base) + tid;
    const float4* dp = reinterpret_cast<const float4*>(src.delta + (uint64_t)row * d + base) + tid;
    float4 a[4], b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) a[j] = __ldcs(gp + j * kThreads);
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = __ldcs(dp + j * kThreads);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      cnt[j] = 4;
      v[j] = add4_rn(a[j], b[j]);
    }
  } else {
    uint64_t ee[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ee[j] = base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = FULL ? 4u : (ee[j] < d ? (uint32_t)min((uint64_t)4, d - ee[j]) : 0u);
    }
    src_load_tile<SRC, 4>(src, row, ee, cnt, v);
  }
  if constexpr (FULL) {
    float4* op = reinterpret_cast<float4*>(out_row + base) + tid;
#pragma unroll
    for (int j = 0; j < 4; ++j) op[j * kThreads] = v[j];
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
      if (cnt[j]) {
        if (src.vec && cnt[j] == 4) {
          *reinterpret_cast<float4*>(out_row + e) = v[j];
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if ((uint32_t)k < cnt[j]) out_row[e + k] = compc(v[j], k);
        }
      }
    }
  }
  if (!marking) return;
  uint32_t ngt[4], ncand[4], idx0[4], keys[16];
  uint32_t kept = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    ngt[j] = 0;
    ncand[j] = 0;
    idx0[j] = (uint32_t)base + (uint32_t)(j * kThreads + tid) * 4u;  // indices fit 32 bits: d < 2^32
    keys[4 * j] = key_of(v[j].x); keys[4 * j + 1] = key_of(v[j].y);
    keys[4 * j + 2] = key_of(v[j].z); keys[4 * j + 3] = key_of(v[j].w);
    if (max(max(keys[4 * j], keys[4 * j + 1]), max(keys[4 * j + 2], keys[4 * j + 3])) >= key_lo) {
      // only the kept entries and the candidates get in here
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (FULL || (uint32_t)k < cnt[j]) {  // entries past the end were loaded as +0 and are no entries
          if (keys[4 * j + k] > key_hi) ngt[j] |= 1u << k;
          else if (keys[4 * j + k] >= key_lo) ncand[j] |= 1u << k;
        }
      }
    }
    kept += __popc(ngt[j]);
  }
  const uint32_t wg = octet_words4(ngt, lane);
  const uint32_t r = lane & 7u;
  if (r < 4) bm_row[(base >> 5) + r * 32u + (tid >> 3)] = wg;
  tile_append(region, s_count, keys, idx0, ncand, lane);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) kept += __shfl_xor_sync(0xffffffffu, kept, o);
  if (lane == 0 && kept) atomicAdd(s_kept, kept);
}

template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1(const SrcParams src, float* v_out, const TopkPred* pred,
                                                         uint32_t* bm_gt, uint64_t bm_stride, uint2* list, uint64_t cap,
                                                         uint2* tile_info, uint64_t ntile) {
  __shared__ uint32_t s_count, s_kept;
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  const uint64_t tile = blockIdx.x, base = tile * kTile;
  const uint64_t d = src.d;
  uint32_t key_lo = 1, key_hi = 0;
  const bool marking = predicted_band(pred, row, &key_lo, &key_hi);
  if (!marking && base >= d) return;  // padding tile and no bitmap to clear
  if (marking) {
    if (tid == 0) { s_count = 0; s_kept = 0; }
    __syncthreads();
  }
  float* out_row = v_out + (uint64_t)row * d;
  uint32_t* bm_row = bm_gt + (uint64_t)row * bm_stride;
  uint2* region = list + (uint64_t)row * cap + base;
  if (src.vec && base + kTile <= d) {
    pass1_tile<SRC, true>(src, row, base, out_row, marking, key_lo, key_hi, bm_row, region, &s_count, &s_kept);
  } else {
    pass1_tile<SRC, false>(src, row, base, out_row, marking, key_lo, key_hi, bm_row, region, &s_count, &s_kept);
  }
  if (marking && base < d) {
    __syncthreads();
    if (tid == 0) tile_info[(uint64_t)row * ntile + tile] = make_uint2(min(s_count, (uint32_t)kTile), s_kept);
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

// Level-1 pick after a miss, one CTA per vector, on the full histogram written by k_topk_hist.
__global__ void __launch_bounds__(1024) k_topk_pick1(uint32_t* hist, TopkState* state, uint32_t k) {
  __shared__ uint32_t s_warp[32], s_out[3];
  const uint32_t tid = threadIdx.x, row = blockIdx.x;
  uint32_t* h = hist + (uint64_t)row * kBins1;
  TopkState* st = state + row;
  if (!st->need_full) return;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; s_out[2] = 0; }
  __syncthreads();
  cta_pick(h, k, s_warp, s_out);
  for (uint32_t b = tid; b < kBins1; b += 1024) h[b] = 0;
  if (tid != 0) return;
  st->tb1 = s_out[0];
  st->k_rem = s_out[1];
  st->need_mark = 1;
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
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k < cnt) comp(v, k) = vrow[e + k];
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
// Bitmap of the entries above the exact threshold bin and the list of those inside it.  A small
// grid strides over the tiles; every bitmap word up to the padded end is written.
__global__ void __launch_bounds__(kThreads) k_topk_mark(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                        uint32_t* bm_gt, uint64_t bm_stride, uint64_t padded, uint2* list,
                                                        uint64_t cap, uint2* tile_info, uint64_t ntile) {
  __shared__ uint32_t s_count;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  if (!state[row].need_mark) return;
  const uint32_t tb = state[row].tb1;
  const float* vrow = v_in + (uint64_t)row * d;
  const uint64_t tiles = padded / kTile;
  for (uint64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const uint64_t base = tile * kTile;
    if (tid == 0) s_count = 0;
    __syncthreads();
    float4 v[4];
    uint32_t cnt[4], idx0[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
      idx0[j] = (uint32_t)e;
      cnt[j] = e < d ? (uint32_t)min((uint64_t)4, d - e) : 0u;
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cnt[j]) {
        if (vec && cnt[j] == 4) {
          v[j] = *reinterpret_cast<const float4*>(vrow + e);
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if ((uint32_t)k < cnt[j]) comp(v[j], k) = vrow[e + k];
        }
      }
    }
    uint32_t ngt[4], ncand[4], keys[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ngt[j] = 0;
      ncand[j] = 0;
      keys[4 * j] = key_of(v[j].x); keys[4 * j + 1] = key_of(v[j].y);
      keys[4 * j + 2] = key_of(v[j].z); keys[4 * j + 3] = key_of(v[j].w);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t bin = keys[4 * j + k] >> 19;
        const bool in = (uint32_t)k < cnt[j];
        ngt[j] |= (in && bin > tb ? 1u : 0u) << k;
        ncand[j] |= (in && bin == tb ? 1u : 0u) << k;
      }
    }
    const uint32_t wg = octet_words4(ngt, lane);
    const uint32_t r = lane & 7u;
    if (r < 4) bm_gt[(uint64_t)row * bm_stride + tile * (kTile / 32) + r * 32u + (tid >> 3)] = wg;
    if (base < d) tile_append(list + (uint64_t)row * cap + base, &s_count, keys, idx0, ncand, lane);
    __syncthreads();
    if (tid == 0 && base < d) tile_info[(uint64_t)row * ntile + tile] = make_uint2(min(s_count, (uint32_t)kTile), 0u);
  }
}

// ---------------------------------------------------------------- tile regions -> dense list
// Copies the candidates out of the per-tile regions into one dense list per vector (order
// irrelevant).  A warp takes eight tiles at a time: one read of their counts, one reservation in
// the dense list for all eight, then the regions.  With HIST the top-12-bit histogram of the keys
// is counted on the way (into s_hist) and the return value is this thread's share of the
// "entries above the band" counts.  Called by whole CTAs.
template <bool HIST>
__device__ __forceinline__ uint32_t gather_tiles(const uint2* lrow, const uint2* info, uint64_t ntile, uint2* drow,
                                                 uint32_t* dense_count, uint32_t* s_hist) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t warps = blockDim.x >> 5;
  uint32_t kept = 0;
  const uint64_t wstep = (uint64_t)gridDim.x * warps * 8;
  for (uint64_t t0 = ((uint64_t)blockIdx.x * warps + (tid >> 5)) * 8; t0 < ntile; t0 += wstep) {
    uint2 mine = make_uint2(0, 0);
    if (lane < 8 && t0 + lane < ntile) mine = info[t0 + lane];
    mine.x = min(mine.x, (uint32_t)kTile);
    kept += mine.y;
    uint32_t incl = mine.x;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= (uint32_t)o) incl += y;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 7);
    if (total == 0) continue;
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(dense_count, total);
    base = __shfl_sync(0xffffffffu, base, 0);
    // the first 32 entries of all eight regions are fetched before any is used
    uint2 first[8];
    uint32_t ns[8], offs[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      ns[u] = __shfl_sync(0xffffffffu, mine.x, u);
      offs[u] = __shfl_sync(0xffffffffu, incl - mine.x, u);
      first[u] = make_uint2(0u, 0u);
      if (lane < ns[u]) first[u] = lrow[(t0 + u) * kTile + lane];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (lane < ns[u]) {
        drow[(uint64_t)base + offs[u] + lane] = first[u];
        if (HIST) atomicAdd(&s_hist[(first[u].x >> 19) & 0xFFFu], 1u);
      }
      const uint2* reg = lrow + (t0 + u) * kTile;
      for (uint32_t i = lane + 32; i < ns[u]; i += 32) {
        const uint2 e = reg[i];
        drow[(uint64_t)base + offs[u] + i] = e;
        if (HIST) atomicAdd(&s_hist[(e.x >> 19) & 0xFFFu], 1u);
      }
    }
  }
  return kept;
}

// After a miss: the list that mark rebuilt, made dense.
__global__ void __launch_bounds__(kThreads) k_topk_compact(const uint2* list, uint64_t cap, const uint2* tile_info,
                                                           uint64_t ntile, uint2* dense, uint32_t* dense_count,
                                                           const TopkState* state) {
  const uint32_t row = blockIdx.y;
  if (!state[row].need_mark) return;
  gather_tiles<false>(list + (uint64_t)row * cap, tile_info + (uint64_t)row * ntile, ntile, dense + (uint64_t)row * cap,
                      &dense_count[row], nullptr);
}

// ---------------------------------------------------------------- list histogram + pick
// One radix digit from the candidate list: LEVEL 1 = key bits 30..19 (and the verdict on the
// prediction), LEVEL 2 = bits 18..7, LEVEL 3 = bits 6..0 (tau and r complete; tau is remembered
// for the next step's prediction).  Several CTAs per vector histogram slices of the list into the
// vector's global histogram; the CTA that finishes last (a ticket counter, no waiting) picks the
// digit and clears histogram and ticket.
template <int LEVEL>
__global__ void __launch_bounds__(1024) k_topk_lhist(const uint2* list, uint64_t cap, const uint2* tile_info, uint64_t ntile,
                                                     uint2* dense, uint32_t* dense_count, uint32_t* kept_count,
                                                     TopkState* state, uint32_t* hist, uint32_t* done, uint32_t k,
                                                     TopkPred* pred) {
  __shared__ uint32_t s_hist[kBins1];
  __shared__ uint32_t s_warp[32], s_out[3];
  __shared__ uint32_t s_last;
  constexpr uint32_t NB = LEVEL == 3 ? 128u : 4096u;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint2* lrow = list + (uint64_t)row * cap;
  const uint2* info = tile_info + (uint64_t)row * ntile;
  TopkState* st = state + row;
  uint32_t band_lo = 1, band_hi = 0;
  // LEVEL 1 reads what pass1 wrote, which exists only if pass1 had a band to work with
  const bool readable = LEVEL != 1 || predicted_band(pred, row, &band_lo, &band_hi);
  const uint32_t tb1 = st->tb1, top24 = (st->tb1 << 12) | st->tb2;
  for (uint32_t b = tid; b < NB; b += 1024) s_hist[b] = 0;
  __syncthreads();
  uint32_t kept = 0;
  if (LEVEL == 1) {
    if (readable) kept = gather_tiles<true>(lrow, info, ntile, dense + (uint64_t)row * cap, &dense_count[row], s_hist);
  } else {
    const uint2* drow = dense + (uint64_t)row * cap;
    const uint64_t n = min((uint64_t)dense_count[row], cap);
    const uint64_t step = (uint64_t)gridDim.x * 8 * 1024;
    for (uint64_t i0 = (uint64_t)blockIdx.x * 8 * 1024; i0 < n; i0 += step) {
      uint32_t key[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint64_t i = i0 + (uint64_t)u * 1024 + tid;
        key[u] = i < n ? drow[i].x : 0xFFFFFFFFu;  // bit 31 set: matches no bin and no prefix
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (LEVEL == 2) {
          if ((key[u] >> 19) == tb1) atomicAdd(&s_hist[(key[u] >> 7) & 0xFFFu], 1u);
        } else {
          if ((key[u] >> 7) == top24) atomicAdd(&s_hist[key[u] & 0x7Fu], 1u);
        }
      }
    }
  }
  if (LEVEL == 1) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kept += __shfl_xor_sync(0xffffffffu, kept, o);
    if (lane == 0 && kept) atomicAdd(&kept_count[row], kept);
  }
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < NB; b += 1024) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&done[row], 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // every CTA of this vector has flushed: read the complete histogram past L1, pick, clear
  for (uint32_t b = tid; b < kBins1; b += 1024) {
    s_hist[b] = b < NB ? __ldcg(&h[b]) : 0u;
    if (b < NB) h[b] = 0;
  }
  uint32_t want = st->k_rem;
  if (LEVEL == 1) {
    const uint32_t kept = __ldcg(&kept_count[row]);
    want = kept < k ? k - kept : 0u;  // 0: the threshold lies above the band
  }
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; s_out[2] = 0; done[row] = 0; }
  __syncthreads();
  cta_pick(s_hist, want, s_warp, s_out);
  if (tid != 0) return;
  if (LEVEL == 1) {
    // the prediction holds iff the k-th largest entry is one of the listed candidates
    uint32_t lo = 1, hi = 0;
    const bool hit = predicted_band(pred, row, &lo, &hi) && want >= 1 && want <= s_out[2];
    if (hit) {
      st->tb1 = s_out[0];
      st->k_rem = s_out[1];
      st->need_full = 0;
      st->need_mark = 0;
    } else {
      st->need_full = 1;  // hist, pick, mark and compact rebuild bitmap and list for the exact bin
      st->need_mark = 1;
      dense_count[row] = 0;
    }
  } else if (LEVEL == 2) {
    st->tb2 = s_out[0];
    st->k_rem = s_out[1];
  } else {
    const uint32_t tau = (top24 << 7) | s_out[0];
    st->tau = tau;
    st->r = s_out[1];
    st->k_rem = s_out[1];
    if (pred) {
      uint32_t lo = 1, hi = 0, centre = 0;
      const bool had = predicted_band(pred, row, &lo, &hi, &centre);
      TopkPred np;
      np.magic = kPredMagic;
      np.tau_prev = had ? pred[row].tau_last : tau;
      np.tau_last = tau;
      if (had) {
        const uint32_t e = tau > centre ? tau - centre : centre - tau;
        const uint32_t old = min(pred[row].err, kMaxErr);
        np.err = min(kMaxErr, max(old - (old >> 2), e));
      } else {
        np.err = kFirstErr;
      }
      pred[row] = np;
    }
  }
}

// ---------------------------------------------------------------- classify
// Candidates above tau join the kept bitmap; candidates equal to tau are set in the tie bitmap
// (which the launcher cleared).  Candidate bits are never set in bm_gt beforehand, so the ORs
// commute with nothing else.
__global__ void __launch_bounds__(kThreads) k_topk_classify(const uint2* dense, const uint32_t* dense_count, uint64_t cap,
                                                            const TopkState* state, uint32_t* bm_gt, uint32_t* bm_tie,
                                                            uint64_t bm_stride) {
  const uint32_t row = blockIdx.y;
  const uint2* drow = dense + (uint64_t)row * cap;
  const uint64_t n = min((uint64_t)dense_count[row], cap);
  const uint32_t tau = state[row].tau;
  uint32_t* g = bm_gt + (uint64_t)row * bm_stride;
  uint32_t* t = bm_tie + (uint64_t)row * bm_stride;
  const uint64_t step = (uint64_t)gridDim.x * kThreads * 4;
  for (uint64_t i0 = (uint64_t)blockIdx.x * kThreads * 4 + threadIdx.x; i0 < n; i0 += step) {
    uint2 e[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t i = i0 + (uint64_t)u * kThreads;
      e[u] = i < n ? drow[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + (uint64_t)u * kThreads >= n) continue;
      if (e[u].x > tau) atomicOr(&g[e[u].y >> 5], 1u << (e[u].y & 31u));
      else if (e[u].x == tau) atomicOr(&t[e[u].y >> 5], 1u << (e[u].y & 31u));
    }
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
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k < cnt[j]) out_row[ee[j] + k] = compc(v[j], k);
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
  #pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k < cnt) comp(v, k) = vrow[e + k];
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

// A scattered 4-byte read: ask L2 to fetch no more than 64 bytes around it.
__device__ __forceinline__ float gather_f32(const float* p) {
  float v;
  asm volatile("ld.global.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
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
  // everything that does not depend on the scan is fetched first, so that a thread has one round
  // of bitmap loads and then up to eight value gathers in flight while the scan runs
  const uint2 pre = seg_pre[(uint64_t)row * nseg + blockIdx.x];
  const uint32_t r = state[row].r;
  const uint4 g4 = *reinterpret_cast<const uint4*>(bm_gt + at);
  const uint4 t4 = *reinterpret_cast<const uint4*>(bm_eq + at);
  const uint32_t gt[4] = {g4.x, g4.y, g4.z, g4.w};
  const uint32_t tie[4] = {t4.x, t4.y, t4.z, t4.w};
  float* vrow = v_io + (uint64_t)row * d;
  // the first two kept entries of every word (ties aside, which are rare and wait for the scan)
  uint32_t b0[4], b1[4];
  float v0[4], v1[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t s0 = gt[i], s1 = s0 & (s0 - 1u);
    b0[i] = s0 ? __ffs(s0) - 1u : 32u;
    b1[i] = s1 ? __ffs(s1) - 1u : 32u;
    v0[i] = b0[i] < 32u ? gather_f32(vrow + (widx + i) * 32u + b0[i]) : 0.f;
    v1[i] = b1[i] < 32u ? gather_f32(vrow + (widx + i) * 32u + b1[i]) : 0.f;
  }
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
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(payload + (uint64_t)row * payload_stride + off_idx);
  float* out_val = reinterpret_cast<float*>(payload + (uint64_t)row * payload_stride + off_val);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (cw[i]) {
      const uint32_t ties_before = pre.y + (excl >> 16);
      uint32_t keep = tie[i];
      const uint32_t room = r > ties_before ? r - ties_before : 0u;
      while ((uint32_t)__popc(keep) > room) keep &= ~(0x80000000u >> __clz(keep));  // drop the highest tie
      uint32_t pos = pre.x + (excl & 0xFFFFu) + min(ties_before, r);
      uint32_t sel = gt[i] | keep;
      if (!keep) {
        // no tie in this word: the prefetched values are its first two entries
        if (b0[i] < 32u) {
          const uint64_t j = (widx + i) * 32u + b0[i];
          if (pos < k) { out_idx[pos] = (uint32_t)j; out_val[pos] = v0[i]; }  // pos < k whenever the counts are consistent
          vrow[j] = 0.f;                                                      // delta = v - Q[v] at a kept entry
          if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, v0[i]));
          ++pos;
        }
        if (b1[i] < 32u) {
          const uint64_t j = (widx + i) * 32u + b1[i];
          if (pos < k) { out_idx[pos] = (uint32_t)j; out_val[pos] = v1[i]; }
          vrow[j] = 0.f;
          if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, v1[i]));
          ++pos;
        }
        sel &= sel - 1u;
        sel &= sel - 1u;  // what is left after the first two (clearing bits of 0 leaves 0)
      }
      while (sel) {
        const uint32_t b = __ffs(sel) - 1u;
        sel &= sel - 1u;
        const uint64_t j = (widx + i) * 32u + b;
        const float val = vrow[j];
        if (pos < k) { out_idx[pos] = (uint32_t)j; out_val[pos] = val; }
        vrow[j] = 0.f;
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
  p->ntile = (d + kTile - 1) / kTile;
  p->list_cap = with_list ? p->ntile * kTile : 0;  // one kTile-slot region per tile
  uint64_t pos = 0;
  p->off_hist = pos;       pos += (uint64_t)rows * kBins1 * 4;      // histogram and list counters are
  p->off_list_count = pos; pos = round16(pos + (uint64_t)rows * 12);  // tickets, kept counts: cleared by one memset
  p->off_state = pos;      pos = round16(pos + (uint64_t)rows * sizeof(TopkState));
  p->off_bm_gt = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_bm_eq = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_seg = pos;        pos = round16(pos + (uint64_t)rows * p->nseg * sizeof(uint2));
  p->off_list = pos;       pos = round16(pos + (uint64_t)rows * p->list_cap * sizeof(uint2));
  p->off_tile_info = pos;  pos = round16(pos + (with_list ? (uint64_t)rows * p->ntile * sizeof(uint2) : 0));
  p->off_dense = pos;      pos = round16(pos + (uint64_t)rows * p->list_cap * sizeof(uint2));
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
  uint2* tile_info = reinterpret_cast<uint2*>(ws + pl.off_tile_info);
  uint2* dense = reinterpret_cast<uint2*>(ws + pl.off_dense);
  const uint64_t d = src.d, cap = pl.list_cap;
  const uint64_t padded = pl.nseg * (uint64_t)kSegElems;
  uint32_t* done = list_count + rows;        // ticket counters of the list histograms
  uint32_t* kept_count = list_count + 2 * rows;  // entries above the predicted band
  cudaError_t e = cudaMemsetAsync(hist, 0, (uint64_t)rows * kBins1 * 4 + (uint64_t)rows * 12, st);
  if (e != cudaSuccess) return e;

  // pass1: one CTA per tile of the padded extent
  const uint64_t ntile_padded = padded / kTile;
  dim3 g1((unsigned)ntile_padded, rows, 1);
  // pass1 without a list keeps its span form
  uint64_t span = 16 * kTile;
  while (span > kTile && ((padded + span - 1) / span) * rows < 148ull * 16ull) span /= 2;
  dim3 g1b((unsigned)((padded + span - 1) / span), rows, 1);
  const uint32_t k32 = (uint32_t)k;
  dim3 gs((unsigned)pl.nseg, rows, 1);
  // kernels that re-read a whole vector after a miss: per vector a grid that (nearly) fills the GPU by
  // itself and strides over the tiles, so that a single vector that missed is not left to a sliver
  // of the machine; the CTAs of the vectors that hit leave at once, so with many vectors the grid
  // per vector is halved to keep those empty launches short
  uint64_t stride_ctas = rows >= 8 ? 148ull * 2ull : 148ull * 4ull;
  if (stride_ctas > padded / kTile) stride_ctas = padded / kTile;
  dim3 gm((unsigned)stride_ctas, rows, 1);

  if (list && k) {
    TopkPred* pred = pl.pred;
#define DSQ_P1(S)                                                                                                 \
  k_topk_pass1<S><<<g1, kThreads, 0, st>>>(src, io.v_inout, pred, bm_gt, pl.bm_stride, list, cap, tile_info, pl.ntile)
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
    dim3 gl((unsigned)(148ull * 2ull / rows ? 148ull * 2ull / rows : 1), rows, 1);
    k_topk_lhist<1><<<gl, 1024, 0, st>>>(list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred);
    k_topk_hist<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, hist);
    k_topk_pick1<<<rows, 1024, 0, st>>>(hist, state, k32);
    k_topk_mark<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, bm_gt, pl.bm_stride, padded, list, cap, tile_info,
                                         pl.ntile);
    k_topk_compact<<<gm, kThreads, 0, st>>>(list, cap, tile_info, pl.ntile, dense, list_count, state);
    k_topk_lhist<2><<<gl, 1024, 0, st>>>(list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred);
    k_topk_lhist<3><<<gl, 1024, 0, st>>>(list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred);
    dim3 gc((unsigned)(148ull * 8ull / rows ? 148ull * 8ull / rows : 1), rows, 1);
    k_topk_classify<<<gc, kThreads, 0, st>>>(dense, list_count, cap, state, bm_gt, bm_eq, pl.bm_stride);
    k_topk_count<<<gs, kThreads, 0, st>>>(bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
    count_launches(11);
  } else {
#define DSQ_P1(S) k_topk_pass1_basic<S><<<g1b, kThreads, 0, st>>>(src, io.v_inout, hist, span)
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
