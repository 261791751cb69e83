// Top-k sparsification (Section 3.2 "Top-k sparsification", Section 5.1 "Top-k compression") fused
// with the error feedback.  Exact selection of the k entries of largest |v| over a whole d-vector,
// ties by lower index, emitted as an index-ordered (index, value) list.
//
// The order of |v| is the order of the bit pattern with the sign cleared (a 31-bit key), so the
// selection is integer work: a radix select finds the key tau of the k-th largest entry and the
// number r of entries equal to tau that still fit.
//
//   pass1     v = source (Eq. 2 / Eq. 4), written over delta; histogram of the top 12 key bits.
//             With a usable history it also marks: two bitmaps (one bit per entry), "certainly
//             kept" (bin above a predicted band of bins) and "candidate" (bin inside the band),
//             and appends the candidates' keys to a dense list.
//   pick      walk the histogram from the top: threshold bin tb, entries still to take inside it;
//             checks that the band pass1 used contains tb
//   mark      only when that check fails (or there was no history): re-read v, write the bitmaps
//             for the exact bin and the candidate keys; otherwise its CTAs leave at once
//   resolve   histogram the next 12 and then the last 7 key bits of the listed candidates: tau, r
//   finalize  bitmaps become key > tau / key == tau (candidate values gathered through the
//             bitmap); per-segment population counts
//   scan      exclusive prefix of the segment counts (per vector)
//   emit      every set bit knows its output slot: write (index, value), zero the entry in delta
//             (delta = v - Q[v], Eq. 3), and on a fused server pass update x at that entry
//
// A wrong, missing or garbage history costs time, never correctness.  No float atomics, no
// spinning; integer histogram atomics commute and output slots come from prefix sums over
// index-ordered bitmaps, so the result does not depend on scheduling.
//
// Without a candidate list (the built-in-scratch entry point keeps its scratch small) the two
// refine kernels gather the candidates through the bitmap instead of reading the list.
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

namespace {

constexpr uint32_t kBins1 = 4096;                  // key bits 30..19
constexpr uint32_t kWordsPerThread = 4;            // finalize / emit / refine: bitmap words per thread
constexpr uint32_t kSegWords = kThreads * kWordsPerThread;  // 1024 bitmap words per segment
constexpr uint32_t kSegElems = kSegWords * 32;     // 32768 entries
constexpr uint64_t kTile = 4096;                   // entries a CTA of pass1 handles per loop trip
constexpr uint32_t kPredMagic = 0x70D1C7EDu;

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

// Band of 12-bit bins expected to contain this step's threshold bin: the last bin, moved by the
// last change (thresholds drift while the error builds up), widened by one bin on each side.
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

// Appends the keys of the entries flagged in sel[j] (bit k = entry k of row j) to the vector's
// candidate list.  One atomic per warp per call; the order inside the list is irrelevant (it is
// only histogrammed).  Called by all 32 lanes.
__device__ __forceinline__ void append_candidates(uint32_t* list_row, uint32_t* count, uint64_t cap,
                                                  const float4 (&v)[4], const uint32_t (&sel)[4], uint32_t lane) {
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
  if (lane == 0) base = atomicAdd(count, total);
  base = __shfl_sync(0xffffffffu, base, 0);
  uint64_t pos = (uint64_t)base + incl - c;
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((sel[j] >> k) & 1u) {
        if (pos < cap) list_row[pos] = key_of(compc(v[j], k));
        ++pos;
      }
}

// ---------------------------------------------------------------- pass1
// span: entries per CTA, a multiple of kTile.  `padded` = bitmap extent in entries (whole segments).
template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1(const SrcParams src, float* v_out, uint32_t* hist, uint64_t span,
                                                         uint64_t padded, const TopkPred* pred, uint32_t* bm_gt,
                                                         uint32_t* bm_eq, uint64_t bm_stride, uint32_t* list,
                                                         uint32_t* list_count, uint64_t cap) {
  __shared__ uint32_t s_hist[kBins1];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  for (uint32_t b = tid; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  uint32_t lo = 1, hi = 0;
  const bool marking = predicted_band(pred, row, &lo, &hi);
  const uint64_t d = src.d;
  const uint64_t begin = (uint64_t)blockIdx.x * span;
  // when marking, the bitmaps are written for whole segments, hence the padded end
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
    uint32_t ngt[4], neq[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ngt[j] = 0;
      neq[j] = 0;
      if (cnt[j]) {
        if (src.vec && cnt[j] == 4) {
          *reinterpret_cast<float4*>(out_row + ee[j]) = v[j];
        } else {
          for (uint32_t k = 0; k < cnt[j]; ++k) out_row[ee[j] + k] = compc(v[j], k);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if ((uint32_t)k < cnt[j]) {
          const uint32_t bin = key_of(compc(v[j], k)) >> 19;
          atomicAdd(&s_hist[bin], 1u);
          ngt[j] |= (bin > hi ? 1u : 0u) << k;
          neq[j] |= (bin >= lo && bin <= hi ? 1u : 0u) << k;
        }
      }
    }
    if (marking) {
      const uint32_t wg = octet_words4(ngt, lane), we = octet_words4(neq, lane);
      const uint32_t r = lane & 7u;
      if (r < 4) {
        const uint64_t w = (uint64_t)row * bm_stride + (base >> 5) + r * 32u + (tid >> 3);
        bm_gt[w] = wg;
        bm_eq[w] = we;
      }
      if (list) append_candidates(list + (uint64_t)row * cap, list_count + row, cap, v, neq, lane);
    }
  }
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < kBins1; b += kThreads) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
}

// ---------------------------------------------------------------- pick
// Called by all 1024 threads of a CTA.  h: 4096 counters (bins above the used range hold 0).
// Finds the bin where the count from the top reaches `want` (1 <= want <= total) and how many
// entries are still to take inside it; result in s_out[0..1] after the final barrier.
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

// One CTA per vector, on the global histogram, which it clears for its next use.
//   level 1: bins = key >> 19            want = k       (also judges the prediction)
//   level 2: bins = (key >> 7) & 0xFFF   want = k_rem   (only without a candidate list)
//   level 3: bins = key & 0x7F           want = k_rem   -> tau and r complete
__global__ void __launch_bounds__(1024) k_topk_pick(uint32_t* hist, TopkState* state, uint32_t level, uint32_t k,
                                                    TopkPred* pred, uint32_t* list_count) {
  __shared__ uint32_t s_warp[32], s_out[2];
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
    // was the band that pass1 marked with right?  If not, the mark kernel has to run.
    uint32_t lo = 1, hi = 0;
    const bool had = predicted_band(pred, row, &lo, &hi);
    const bool hit = had && tb >= lo && tb <= hi;
    st->need_mark = hit ? 0u : 1u;
    if (!hit && list_count) list_count[row] = 0;  // mark will list the candidates afresh
    if (pred) {
      TopkPred np;
      np.magic = kPredMagic;
      np.tb_prev = had ? pred[row].tb_last : tb;
      np.tb_last = tb;
      np.pad = 0;
      pred[row] = np;
    }
  } else if (level == 2) {
    st->tb2 = tb;
  } else {
    st->tau = (st->tb1 << 19) | (st->tb2 << 7) | tb;
    st->r = rem;
  }
}

// ---------------------------------------------------------------- mark
// Runs only for vectors whose prediction missed (or had none): bitmaps for the exact threshold
// bin, bin > tb / bin == tb, and the candidate keys.  One 8192-entry block per loop trip over a
// small grid; every bitmap word up to the padded end is written.
__global__ void __launch_bounds__(kThreads) k_topk_mark(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                        uint32_t* bm_gt, uint32_t* bm_eq, uint64_t bm_stride,
                                                        uint64_t padded, uint32_t* list, uint32_t* list_count,
                                                        uint64_t cap) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  if (!state[row].need_mark) return;
  const uint32_t tb = state[row].tb1;
  const float* vrow = v_in + (uint64_t)row * d;
  const uint64_t nblk = padded / 8192;
  for (uint64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
    const uint64_t blk_base = blk * 8192;
    float4 v[8];
    uint32_t cnt[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint64_t e = blk_base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = e < d ? (uint32_t)min((uint64_t)4, d - e) : 0u;
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cnt[j]) {
        if (vec && cnt[j] == 4) {
          v[j] = *reinterpret_cast<const float4*>(vrow + e);
        } else {
          for (uint32_t k = 0; k < cnt[j]; ++k) comp(v[j], k) = vrow[e + k];
        }
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t ngt[4], neq[4];
      float4 vh[4];
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int j = h * 4 + jj;
        vh[jj] = v[j];
        ngt[jj] = 0;
        neq[jj] = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t bin = key_of(compc(v[j], k)) >> 19;
          const bool in = (uint32_t)k < cnt[j];
          ngt[jj] |= (in && bin > tb ? 1u : 0u) << k;
          neq[jj] |= (in && bin == tb ? 1u : 0u) << k;
        }
      }
      const uint32_t wg = octet_words4(ngt, lane), we = octet_words4(neq, lane);
      const uint32_t r = lane & 7u;
      if (r < 4) {
        const uint64_t w = (uint64_t)row * bm_stride + (blk_base >> 5) + (uint32_t)((h * 4 + r) * 32) + (tid >> 3);
        bm_gt[w] = wg;
        bm_eq[w] = we;
      }
      if (list) append_candidates(list + (uint64_t)row * cap, list_count + row, cap, vh, neq, lane);
    }
  }
}

// ---------------------------------------------------------------- resolve
// One CTA per vector: the second and third radix digits from the candidate list.
__global__ void __launch_bounds__(1024) k_topk_resolve(const uint32_t* list, const uint32_t* list_count, uint64_t cap,
                                                       TopkState* state) {
  __shared__ uint32_t s_hist[kBins1];
  __shared__ uint32_t s_warp[32], s_out[2];
  const uint32_t tid = threadIdx.x, row = blockIdx.x;
  const uint32_t* lrow = list + (uint64_t)row * cap;
  const uint64_t n = min((uint64_t)list_count[row], cap);
  TopkState* st = state + row;
  const uint32_t tb1 = st->tb1, want = st->k_rem;
  for (uint32_t b = tid; b < kBins1; b += 1024) s_hist[b] = 0;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; }
  __syncthreads();
  for (uint64_t i = tid; i < n; i += 1024) {
    const uint32_t key = lrow[i];
    if ((key >> 19) == tb1) atomicAdd(&s_hist[(key >> 7) & 0xFFFu], 1u);
  }
  __syncthreads();
  cta_pick(s_hist, want, s_warp, s_out);
  const uint32_t tb2 = s_out[0], rem2 = s_out[1];
  __syncthreads();
  for (uint32_t b = tid; b < kBins1; b += 1024) s_hist[b] = 0;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; }
  __syncthreads();
  const uint32_t top24 = (tb1 << 12) | tb2;
  for (uint64_t i = tid; i < n; i += 1024) {
    const uint32_t key = lrow[i];
    if ((key >> 7) == top24) atomicAdd(&s_hist[key & 0x7Fu], 1u);
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

// ---------------------------------------------------------------- refine (no candidate list)
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
  const uint32_t top = state[row].tb1, top24 = (state[row].tb1 << 12) | state[row].tb2;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t w = ws[i];
    while (w) {
      const uint32_t b = __ffs(w) - 1u;
      w &= w - 1u;
      const uint32_t key = key_of(vrow[(widx + i) * 32u + b]);
      if (LEVEL == 2) {
        if ((key >> 19) == top) atomicAdd(&s_hist[(key >> 7) & 0xFFFu], 1u);
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

// ---------------------------------------------------------------- finalize
// bm_gt <- key > tau, bm_eq <- key == tau; population counts per segment (x: gt, y: ties).
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

// ---------------------------------------------------------------- scan
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

// ---------------------------------------------------------------- emit
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
  // exclusive scan inside the segment; gt count in the low 16 bits, tie count in the high 16
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
  p->list_cap = with_list ? (d + 3) / 4 * 4 : 0;
  uint64_t pos = 0;
  p->off_hist = pos;       pos += (uint64_t)rows * kBins1 * 4;      // histogram and list counters are
  p->off_list_count = pos; pos = round16(pos + (uint64_t)rows * 4);  // cleared by one memset
  p->off_state = pos;      pos = round16(pos + (uint64_t)rows * sizeof(TopkState));
  p->off_bm_gt = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_bm_eq = pos;      pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_seg = pos;        pos = round16(pos + (uint64_t)rows * p->nseg * sizeof(uint2));
  p->off_list = pos;       pos = round16(pos + (uint64_t)rows * p->list_cap * 4);
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
  uint32_t* bm_eq = reinterpret_cast<uint32_t*>(ws + pl.off_bm_eq);
  uint2* seg = reinterpret_cast<uint2*>(ws + pl.off_seg);
  uint32_t* list = pl.list_cap ? reinterpret_cast<uint32_t*>(ws + pl.off_list) : nullptr;
  const uint64_t d = src.d, cap = pl.list_cap;
  const uint64_t padded = pl.nseg * (uint64_t)kSegElems;
  cudaError_t e = cudaMemsetAsync(hist, 0, (uint64_t)rows * kBins1 * 4 + (uint64_t)rows * 4, st);
  if (e != cudaSuccess) return e;

  // entries per CTA: long spans amortise the histogram flush, but the grid must still fill the GPU
  uint64_t span = 16 * kTile;
  while (span > 2 * kTile && ((padded + span - 1) / span) * rows < 148ull * 16ull) span /= 2;
  dim3 g1((unsigned)((padded + span - 1) / span), rows, 1);
  TopkPred* pred = k ? pl.pred : nullptr;
#define DSQ_P1(S)                                                                                                        \
  k_topk_pass1<S><<<g1, kThreads, 0, st>>>(src, io.v_inout, hist, span, padded, pred, bm_gt, bm_eq, pl.bm_stride, list, \
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
  count_launches(1);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if (k == 0) return cudaSuccess;  // nothing kept: Q[v] = 0, delta = v, x unchanged

  const uint32_t k32 = (uint32_t)k;
  dim3 gs((unsigned)pl.nseg, rows, 1);
  // the mark kernel normally has nothing to do: a small grid that strides over the blocks
  uint64_t mark_ctas = 148ull * 8ull / rows;
  if (mark_ctas < 1) mark_ctas = 1;
  if (mark_ctas > padded / 8192) mark_ctas = padded / 8192;
  dim3 gm((unsigned)mark_ctas, rows, 1);
  k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 1, k32, pred, list ? list_count : nullptr);
  k_topk_mark<<<gm, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, bm_gt, bm_eq, pl.bm_stride, padded, list, list_count,
                                       cap);
  if (list) {
    k_topk_resolve<<<rows, 1024, 0, st>>>(list, list_count, cap, state);
    count_launches(3);
  } else {
    k_topk_refine<2><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 2, k32, nullptr, nullptr);
    k_topk_refine<3><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 3, k32, nullptr, nullptr);
    count_launches(6);
  }
  k_topk_finalize<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
  k_topk_scan<<<rows, 1024, 0, st>>>(seg, pl.nseg, state, k32, io.dev_status);
  k_topk_emit<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg,
                                       reinterpret_cast<uint8_t*>(io.idx), io.payload_stride, 0,
                                       (uint64_t)(reinterpret_cast<uint8_t*>(io.val) - reinterpret_cast<uint8_t*>(io.idx)),
                                       k32, io.x, io.gamma);
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace dsq
