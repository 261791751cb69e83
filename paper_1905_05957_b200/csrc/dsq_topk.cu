// Top-k sparsification (Section 3.2 "Top-k sparsification", Section 5.1 "Top-k compression") fused
// with the error feedback.  Exact selection of the k entries of largest |v| over a whole d-vector,
// ties by lower index, emitted as an index-ordered (index, value) list.
//
// The order of |v| is the order of the bit pattern with the sign cleared (a 31-bit key), so the
// selection is integer work: a radix select finds the key tau of the k-th largest entry and the
// number r of entries equal to tau that still fit.
//
//   pass1     v = source (Eq. 2 / Eq. 4), written over delta; histogram of the top 12 key bits
//   pick      walk the histogram from the top: threshold bin tb, entries still to take
//   mark      re-read v once; two bitmaps (one bit per entry): bin > tb, bin == tb (candidates)
//   refine x2 histogram the next 12, then the last 7 key bits of the candidates (gathered through
//             the candidate bitmap), pick after each: tau and r are known
//   finalize  bitmaps become: key > tau, key == tau; per-segment population counts
//   scan      exclusive prefix of the segment counts (per vector)
//   emit      every set bit knows its output slot: write (index, value), zero the entry in delta
//             (delta = v - Q[v], Eq. 3), and on a fused server pass update x at that entry
//
// No float atomics, no spinning, and the result does not depend on scheduling: integer histogram
// atomics commute, and output slots come from prefix sums over index-ordered bitmaps.
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

namespace {

constexpr uint32_t kBins1 = 4096;        // key bits 30..19
constexpr uint32_t kSegWords = 256;      // bitmap words per segment (one per thread)
constexpr uint32_t kSegElems = kSegWords * 32;
constexpr uint64_t kPass1Step = 4096;    // entries one CTA of pass1 handles per loop trip

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

// ---------------------------------------------------------------- pass1
template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1(const SrcParams src, float* v_out, uint32_t* hist, uint64_t span) {
  __shared__ uint32_t s_hist[kBins1];
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  for (uint32_t b = tid; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  const uint64_t d = src.d;
  const uint64_t begin = (uint64_t)blockIdx.x * span;  // span: a multiple of kPass1Step
  const uint64_t end = min(begin + span, d);
  float* out_row = v_out + (uint64_t)row * d;
  for (uint64_t base = begin; base < end; base += kPass1Step) {
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
      const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
      if (src.vec && cnt[j] == 4) {
        *reinterpret_cast<float4*>(out_row + e) = v[j];
      } else {
        for (uint32_t k = 0; k < cnt[j]; ++k) out_row[e + k] = compc(v[j], k);
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

// ---------------------------------------------------------------- pick
// One CTA per vector.  Finds the bin where the count from the top reaches `want`, records it and
// the number still to take inside it, then clears the histogram for its next use.
//   level 1: bins = key >> 19            want = k
//   level 2: bins = (key >> 7) & 0xFFF   want = k_rem
//   level 3: bins = key & 0x7F           want = k_rem   -> tau and r complete
__global__ void __launch_bounds__(1024) k_topk_pick(uint32_t* hist, TopkState* state, uint32_t level, uint32_t k) {
  __shared__ uint32_t s_warp[32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5;
  const uint32_t row = blockIdx.x;
  uint32_t* h = hist + (uint64_t)row * kBins1;
  TopkState* st = state + row;
  const uint32_t want = level == 1 ? k : st->k_rem;
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
    uint32_t w = s_warp[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= (uint32_t)o) wi += y;
    }
    s_warp[lane] = wi - w;  // exclusive prefix of the warp totals
  }
  __syncthreads();
  const uint32_t above = s_warp[wrp] + incl - mine;  // entries in bins above this thread's four
  h[b0] = 0; h[b0 + 1] = 0; h[b0 + 2] = 0; h[b0 + 3] = 0;
  if (want > above && want <= above + mine) {
    uint32_t cum = above, tb = b0 + 3;
    const uint32_t cs[4] = {c3, c2, c1, c0};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (want <= cum + cs[i]) { tb = b0 + 3 - i; break; }
      cum += cs[i];
    }
    const uint32_t rem = want - cum;
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
}

// ---------------------------------------------------------------- mark
// One segment (8192 entries, 256 bitmap words) per CTA.  Bitmap rows are padded to whole segments
// and every word of the segment is written, so later kernels never meet stale words.
__global__ void __launch_bounds__(kThreads) k_topk_mark(const float* v_in, uint64_t d, int vec, const TopkState* state,
                                                        uint32_t* bm_gt, uint32_t* bm_eq, uint64_t bm_stride) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint32_t tb = state[row].tb1;
  const float* vrow = v_in + (uint64_t)row * d;
  const uint64_t seg_base = (uint64_t)blockIdx.x * kSegElems;
  float4 v[8];
  uint32_t cnt[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint64_t e = seg_base + (uint64_t)(j * kThreads + tid) * 4u;
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
  for (int j = 0; j < 8; ++j) {
    uint32_t ngt = 0, neq = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t bin = key_of(compc(v[j], k)) >> 19;
      const bool in = (uint32_t)k < cnt[j];
      ngt |= (in && bin > tb ? 1u : 0u) << k;
      neq |= (in && bin == tb ? 1u : 0u) << k;
    }
    uint32_t wg = ngt << ((lane & 7u) * 4u), we = neq << ((lane & 7u) * 4u);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      wg |= __shfl_xor_sync(0xffffffffu, wg, o);
      we |= __shfl_xor_sync(0xffffffffu, we, o);
    }
    if ((lane & 7u) == 0) {
      const uint64_t w = (uint64_t)row * bm_stride + (uint64_t)blockIdx.x * kSegWords + (uint32_t)(j * 32) + (tid >> 3);
      bm_gt[w] = wg;
      bm_eq[w] = we;
    }
  }
}

// ---------------------------------------------------------------- refine
// Histogram of the next key digit over the candidates (set bits of bm_eq), values gathered from v.
template <int LEVEL>
__global__ void __launch_bounds__(kThreads) k_topk_refine(const float* v_in, uint64_t d, const TopkState* state,
                                                          const uint32_t* bm_eq, uint64_t bm_stride, uint32_t* hist) {
  constexpr uint32_t NB = LEVEL == 2 ? 4096u : 128u;
  __shared__ uint32_t s_hist[NB];
  __shared__ uint32_t s_any;
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid;
  uint32_t w = bm_eq[(uint64_t)row * bm_stride + widx];
  if (tid == 0) s_any = 0;
  __syncthreads();
  if (w) s_any = 1;
  __syncthreads();
  if (!s_any) return;  // uniform: no candidate in this segment
  for (uint32_t b = tid; b < NB; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  const float* vrow = v_in + (uint64_t)row * d;
  const uint32_t mid = state[row].tb2;
  while (w) {
    const uint32_t b = __ffs(w) - 1u;
    w &= w - 1u;
    const uint32_t key = key_of(vrow[widx * 32u + b]);
    if (LEVEL == 2) {
      atomicAdd(&s_hist[(key >> 7) & 0xFFFu], 1u);
    } else if (((key >> 7) & 0xFFFu) == mid) {
      atomicAdd(&s_hist[key & 0x7Fu], 1u);
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
// bm_gt <- key > tau, bm_eq <- key == tau; population counts per segment (low half: gt, high: ties).
__global__ void __launch_bounds__(kThreads) k_topk_finalize(const float* v_in, uint64_t d, const TopkState* state,
                                                            uint32_t* bm_gt, uint32_t* bm_eq, uint64_t bm_stride,
                                                            uint2* seg_cnt, uint64_t nseg) {
  __shared__ uint32_t s_gt[kThreads / 32], s_tie[kThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid;
  const uint64_t at = (uint64_t)row * bm_stride + widx;
  uint32_t gt = bm_gt[at], cand = bm_eq[at], tie = 0;
  if (cand) {
    const float* vrow = v_in + (uint64_t)row * d;
    const uint32_t tau = state[row].tau;
    while (cand) {
      const uint32_t b = __ffs(cand) - 1u;
      cand &= cand - 1u;
      const uint32_t key = key_of(vrow[widx * 32u + b]);
      if (key > tau) gt |= 1u << b;
      else if (key == tau) tie |= 1u << b;
    }
    bm_gt[at] = gt;
  }
  bm_eq[at] = tie;
  uint32_t ng = __popc(gt), nt = __popc(tie);
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
  const uint64_t widx = (uint64_t)blockIdx.x * kSegWords + tid;
  const uint64_t at = (uint64_t)row * bm_stride + widx;
  const uint32_t gt = bm_gt[at], tie = bm_eq[at];
  // exclusive scan inside the segment; gt count in the low 16 bits, tie count in the high 16
  const uint32_t mine = __popc(gt) | (__popc(tie) << 16);
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
  const uint32_t excl = warp_pre + incl - mine;
  if (!(gt | tie)) return;
  const uint2 pre = seg_pre[(uint64_t)row * nseg + blockIdx.x];
  const uint32_t r = state[row].r;
  const uint32_t ties_before = pre.y + (excl >> 16);
  uint32_t keep = tie;
  const uint32_t room = r > ties_before ? r - ties_before : 0u;
  while ((uint32_t)__popc(keep) > room) keep &= ~(0x80000000u >> __clz(keep));  // drop the highest tie
  uint32_t sel = gt | keep;
  uint32_t pos = pre.x + (excl & 0xFFFFu) + min(ties_before, r);
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(payload + (uint64_t)row * payload_stride + off_idx);
  float* out_val = reinterpret_cast<float*>(payload + (uint64_t)row * payload_stride + off_val);
  float* vrow = v_io + (uint64_t)row * d;
  while (sel) {
    const uint32_t b = __ffs(sel) - 1u;
    sel &= sel - 1u;
    const uint64_t j = widx * 32u + b;
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

}  // namespace

void topk_plan(uint64_t d, uint32_t rows, uint64_t k, TopkPlan* p) {
  p->d = d;
  p->rows = rows;
  p->k = k;
  const uint64_t nw = (d + 31) / 32;
  p->nseg = (nw + kSegWords - 1) / kSegWords;
  p->bm_stride = p->nseg * kSegWords;
  uint64_t pos = 0;
  p->off_hist = pos;  pos = round16(pos + (uint64_t)rows * kBins1 * 4);
  p->off_state = pos; pos = round16(pos + (uint64_t)rows * sizeof(TopkState));
  p->off_bm_gt = pos; pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_bm_eq = pos; pos = round16(pos + (uint64_t)rows * p->bm_stride * 4);
  p->off_seg = pos;   pos = round16(pos + (uint64_t)rows * p->nseg * sizeof(uint2));
  p->bytes = pos;
}

cudaError_t launch_topk(int srck, const SrcParams& src, const TopkPlan& pl, void* workspace, const TopkIO& io,
                        uint32_t rows, uint64_t k, cudaStream_t st) {
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + pl.off_hist);
  TopkState* state = reinterpret_cast<TopkState*>(ws + pl.off_state);
  uint32_t* bm_gt = reinterpret_cast<uint32_t*>(ws + pl.off_bm_gt);
  uint32_t* bm_eq = reinterpret_cast<uint32_t*>(ws + pl.off_bm_eq);
  uint2* seg = reinterpret_cast<uint2*>(ws + pl.off_seg);
  const uint64_t d = src.d;
  cudaError_t e = cudaMemsetAsync(hist, 0, (uint64_t)rows * kBins1 * 4, st);
  if (e != cudaSuccess) return e;

  // entries per CTA: long spans amortise the histogram flush, but the grid must still fill the GPU
  uint64_t span = 16 * kPass1Step;
  while (span > kPass1Step && ((d + span - 1) / span) * rows < 148ull * 16ull) span /= 2;
  dim3 g1((unsigned)((d + span - 1) / span), rows, 1);
#define DSQ_P1(S) k_topk_pass1<S><<<g1, kThreads, 0, st>>>(src, io.v_inout, hist, span)
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
  k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 1, k32);
  k_topk_mark<<<gs, kThreads, 0, st>>>(io.v_inout, d, src.vec, state, bm_gt, bm_eq, pl.bm_stride);
  k_topk_refine<2><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
  k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 2, k32);
  k_topk_refine<3><<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
  k_topk_pick<<<rows, 1024, 0, st>>>(hist, state, 3, k32);
  k_topk_finalize<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
  k_topk_scan<<<rows, 1024, 0, st>>>(seg, pl.nseg, state, k32, io.dev_status);
  k_topk_emit<<<gs, kThreads, 0, st>>>(io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg,
                                       reinterpret_cast<uint8_t*>(io.idx), io.payload_stride, 0,
                                       (uint64_t)(reinterpret_cast<uint8_t*>(io.val) - reinterpret_cast<uint8_t*>(io.idx)),
                                       k32, io.x, io.gamma);
  count_launches(10);
  return cudaGetLastError();
}

}  // namespace dsq
