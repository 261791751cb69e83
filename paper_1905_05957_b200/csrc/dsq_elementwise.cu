// Elementwise kernels: Q = identity (Algorithm 1 then is parallel SGD, Section 1), the stand-alone
// model update x = x - gamma Q[v] (Algorithm 1, last line of the loop), and the ordered
// accumulation of sparse worker payloads for the server mean (first line of Eq. 4).
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

// Whether a pass writes a residual: a worker with error feedback always does, a worker without
// compensation never, a server pass when it was given a destination.
template <int SRC>
__device__ __forceinline__ bool keeps_error(const float* delta_out) {
  return SRC != SRC_WORKER_PLAIN && (SRC == SRC_WORKER || delta_out != nullptr);
}

template <int SRC>
__global__ void __launch_bounds__(kThreads) k_identity(const SrcParams src, float* out_c, uint64_t c_row_stride,
                                                       float* delta_out, uint64_t delta_row_stride, float* x,
                                                       float gamma) {
  pdl_prologue();
  const uint32_t row = blockIdx.y;
  const uint64_t nq = (src.d + 3) / 4;
  // the loop bound is the same for all threads of the CTA: the source is read warp-cooperatively
  for (uint64_t q0 = (uint64_t)blockIdx.x * kThreads; q0 < nq; q0 += (uint64_t)gridDim.x * kThreads) {
    const uint64_t ee[1] = {(q0 + threadIdx.x) * 4};
    const uint64_t e = ee[0];
    const uint32_t cc[1] = {e < src.d ? (uint32_t)min((uint64_t)4, src.d - e) : 0u};
    const uint32_t cnt = cc[0];
    float4 vv[1];
    src_load_tile<SRC, 1>(src, row, ee, cc, vv);
    const float4 v = vv[0];
    if (!cnt) continue;
    store_row4(out_c + (uint64_t)row * c_row_stride, e, cnt, 1, v);  // Q[v] = v
    if (keeps_error<SRC>(delta_out)) store_row4(delta_out + (uint64_t)row * delta_row_stride, e, cnt, src.vec, make_float4(0.f, 0.f, 0.f, 0.f));
    if (x) {
      float4 xv = load_row4(x, e, cnt, 1);
      xv.x = __fsub_rn(xv.x, __fmul_rn(gamma, v.x)); xv.y = __fsub_rn(xv.y, __fmul_rn(gamma, v.y));
      xv.z = __fsub_rn(xv.z, __fmul_rn(gamma, v.z)); xv.w = __fsub_rn(xv.w, __fmul_rn(gamma, v.w));
      store_row4(x, e, cnt, 1, xv);
    }
  }
}

static unsigned grid_for(uint64_t items) {
  const uint64_t blocks = (items + kThreads - 1) / kThreads;
  const uint64_t cap = 148ull * 8ull * 4ull;  // a few waves of 8 CTAs on each of the 148 SMs
  return (unsigned)(blocks < cap ? (blocks ? blocks : 1) : cap);
}

cudaError_t launch_identity(int srck, const SrcParams& src, float* out_c, uint64_t c_row_stride, float* delta_out,
                            uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st) {
  dim3 grid(grid_for((src.d + 3) / 4), rows, 1);
#define DSQ_ID(S) launch_pdl(k_identity<S>, grid, kThreads, st, src, out_c, c_row_stride, delta_out, delta_row_stride, x, gamma)
  DSQ_SWITCH_SRC(srck, DSQ_ID)
#undef DSQ_ID
  count_launches(1);
  return cudaGetLastError();
}

// Q = clipping (Section 3.2): the low BITS bits of every number are set to zero; the payload is what
// is left, bits(v) >> BITS, as 16- or 8-bit entries.  The residual v - Q[v] is exact.
template <int SRC, int BITS>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm)
k_clip(const SrcParams src, uint8_t* out_hi, uint64_t hi_row_stride, float* delta_out, uint64_t delta_row_stride, float* x,
       float gamma) {
  pdl_prologue();
  constexpr uint32_t kMask = 0xFFFFFFFFu << BITS;
  const uint32_t row = blockIdx.y;
  const uint64_t nq = (src.d + 3) / 4;
  uint8_t* hi = out_hi + (uint64_t)row * hi_row_stride;
  // the loop bound is the same for all threads of the CTA: the source is read warp-cooperatively
  for (uint64_t q0 = (uint64_t)blockIdx.x * kThreads; q0 < nq; q0 += (uint64_t)gridDim.x * kThreads) {
    const uint64_t ee[1] = {(q0 + threadIdx.x) * 4};
    const uint64_t e = ee[0];
    const uint32_t cc[1] = {e < src.d ? (uint32_t)min((uint64_t)4, src.d - e) : 0u};
    const uint32_t cnt = cc[0];
    float4 vv[1];
    src_load_tile<SRC, 1>(src, row, ee, cc, vv);
    const float4 v = vv[0];
    if (!cnt) continue;
    const uint32_t u0 = __float_as_uint(v.x), u1 = __float_as_uint(v.y), u2 = __float_as_uint(v.z), u3 = __float_as_uint(v.w);
    const float4 C = make_float4(__uint_as_float(u0 & kMask), __uint_as_float(u1 & kMask), __uint_as_float(u2 & kMask),
                                 __uint_as_float(u3 & kMask));
    if (cnt == 4) {
      if (BITS == 16) {
        __stcs(reinterpret_cast<uint2*>(hi + 2 * e), make_uint2(u0 >> 16 | (u1 & kMask), u2 >> 16 | (u3 & kMask)));
      } else {
        __stcs(reinterpret_cast<uint32_t*>(hi + e), u0 >> 24 | (u1 >> 24) << 8 | (u2 >> 24) << 16 | (u3 & kMask));
      }
    } else {
      const uint32_t us[4] = {u0, u1, u2, u3};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if ((uint32_t)k < cnt) {
          if (BITS == 16) reinterpret_cast<uint16_t*>(hi + 2 * e)[k] = (uint16_t)(us[k] >> 16);
          else hi[e + k] = (uint8_t)(us[k] >> 24);
        }
      }
    }
    if (keeps_error<SRC>(delta_out)) store_row4(delta_out + (uint64_t)row * delta_row_stride, e, cnt, src.vec, sub4_rn(v, C));  // Eq. 3 / Eq. 4
    if (x) {
      float4 xv = load_row4(x, e, cnt, 1);
      xv.x = __fsub_rn(xv.x, __fmul_rn(gamma, C.x)); xv.y = __fsub_rn(xv.y, __fmul_rn(gamma, C.y));
      xv.z = __fsub_rn(xv.z, __fmul_rn(gamma, C.z)); xv.w = __fsub_rn(xv.w, __fmul_rn(gamma, C.w));
      store_row4(x, e, cnt, 1, xv);
    }
  }
}

template <int BITS>
static cudaError_t launch_clip_bits(int srck, const SrcParams& src, uint8_t* out_hi, uint64_t hi_row_stride, float* delta_out,
                                    uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st) {
  dim3 grid(grid_for((src.d + 3) / 4), rows, 1);
#define DSQ_CL(S) launch_pdl(k_clip<S, BITS>, grid, kThreads, st, src, out_hi, hi_row_stride, delta_out, delta_row_stride, x, gamma)
  DSQ_SWITCH_SRC(srck, DSQ_CL)
#undef DSQ_CL
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_clip(int srck, const SrcParams& src, uint32_t bits, uint8_t* out_hi, uint64_t hi_row_stride,
                        float* delta_out, uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st) {
  if (bits == 16) return launch_clip_bits<16>(srck, src, out_hi, hi_row_stride, delta_out, delta_row_stride, x, gamma, rows, st);
  if (bits == 24) return launch_clip_bits<24>(srck, src, out_hi, hi_row_stride, delta_out, delta_row_stride, x, gamma, rows, st);
  return cudaErrorInvalidValue;
}

// The draw of every chunk of every vector of a pass, straight into the payload: o = first Philox word
// of counter (0xFFFFFFFF, chunk, worker or 0xFFFFFFFF on the server pass, step), mod S.
// The CTA that holds the last chunk also stores +0 into the value slots of the positions wholly past
// d (a short last chunk): no entry ever lands there, and the payload must not depend on what the
// buffer held before.
__global__ void __launch_bounds__(kThreads) k_rsparse_draw(const RsparseParams rp, uint64_t nc, uint64_t d) {
  pdl_prologue();
  const uint32_t row = blockIdx.y;
  const uint64_t c = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  if (c < nc) {
    const uint4 rnd = philox4x32_10(make_uint4(0xFFFFFFFFu, (uint32_t)c + rp.chunk0, rp.server_pass ? 0xFFFFFFFFu : row + rp.row0, rp.step),
                                    rp.keys);
    rp.out_off[(uint64_t)row * rp.off_stride + c] = rnd.x & ((1u << rp.log2_keep) - 1u);
  }
  if (blockIdx.x == gridDim.x - 1) {
    const uint64_t slots = nc << (rp.log2_chunk - rp.log2_keep);
    float* val = rp.out_val + (uint64_t)row * rp.val_stride;
    for (uint64_t s = ((d - 1) >> rp.log2_keep) + 1 + threadIdx.x; s < slots; s += kThreads) val[s] = 0.f;
  }
}

// Q = randomised sparsification (Section 3.2): the entries of a chunk share one draw o in 0..S-1 and
// the entry at offset t survives iff t mod S == o; survivors go to slot j / S of the payload.
template <int SRC>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm)
k_rsparse(const SrcParams src, const RsparseParams rp, float* delta_out, uint64_t delta_row_stride, float* x, float gamma) {
  pdl_prologue();
  const uint32_t row = blockIdx.y;
  const uint64_t nq = (src.d + 3) / 4;
  const uint32_t smask = (1u << rp.log2_keep) - 1u;
  const float factor = rp.scaled ? (float)(1u << rp.log2_keep) : 1.0f;
  float* val = rp.out_val + (uint64_t)row * rp.val_stride;
  const uint32_t* off = rp.out_off + (uint64_t)row * rp.off_stride;
  // one float4 per thread and trip (two on the server passes measured slower: the decode of n payloads
  // already fills the 64 registers that four resident CTAs allow)
  constexpr int V = 1;
  // the loop bound is the same for all threads of the CTA: the source is read warp-cooperatively
  for (uint64_t q0 = (uint64_t)blockIdx.x * kThreads * V; q0 < nq; q0 += (uint64_t)gridDim.x * kThreads * V) {
    uint64_t ee[V];
    uint32_t cc[V], oo[V];
    float4 vv[V], xx[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
      ee[j] = (q0 + (uint64_t)j * kThreads + threadIdx.x) * 4;
      cc[j] = ee[j] < src.d ? (uint32_t)min((uint64_t)4, src.d - ee[j]) : 0u;
      oo[j] = cc[j] ? __ldg(off + (ee[j] >> rp.log2_chunk)) : 0u;  // the chunk's draw, made by k_rsparse_draw
      xx[j] = (x && cc[j]) ? load_row4(x, ee[j], cc[j], 1) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    src_load_tile<SRC, V>(src, row, ee, cc, vv);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      const uint64_t e = ee[j];
      const uint32_t cnt = cc[j], o = oo[j];
      const float4 v = vv[j];
      if (!cnt) continue;
      float4 C = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if ((uint32_t)k < cnt && (((uint32_t)e + k) & smask) == o) {
          const float kept = __fmul_rn(factor, compc(v, k));
          comp(C, k) = kept;
          val[(e + k) >> rp.log2_keep] = kept;
        }
      }
      // the group of S positions that holds the last entry: if its survivor lies past the end, its slot
      // is sent as +0 (it may still hold a survivor of an earlier step); the slots of the groups
      // wholly past the end are cleared by k_rsparse_draw
      if (e + cnt == src.d) {
        const uint64_t group = (src.d - 1) >> rp.log2_keep;
        if ((group << rp.log2_keep) + o >= src.d) val[group] = 0.f;
      }
      if (keeps_error<SRC>(delta_out)) store_row4(delta_out + (uint64_t)row * delta_row_stride, e, cnt, src.vec, sub4_rn(v, C));  // Eq. 3 / Eq. 4
      if (x) {
        float4 xv = xx[j];
        xv.x = __fsub_rn(xv.x, __fmul_rn(gamma, C.x)); xv.y = __fsub_rn(xv.y, __fmul_rn(gamma, C.y));
        xv.z = __fsub_rn(xv.z, __fmul_rn(gamma, C.z)); xv.w = __fsub_rn(xv.w, __fmul_rn(gamma, C.w));
        store_row4(x, e, cnt, 1, xv);
      }
    }
  }
}

cudaError_t launch_rsparse(int srck, const SrcParams& src, const RsparseParams& rp, float* delta_out, uint64_t delta_row_stride,
                           float* x, float gamma, uint32_t rows, cudaStream_t st) {
  const uint64_t nc = (src.d + (1ull << rp.log2_chunk) - 1) >> rp.log2_chunk;
  launch_pdl(k_rsparse_draw, dim3((unsigned)((nc + kThreads - 1) / kThreads), rows, 1), kThreads, st, rp, nc, src.d);
  count_launches(1);
  dim3 grid(grid_for((src.d + 3) / 4), rows, 1);
#define DSQ_RS(S) launch_pdl(k_rsparse<S>, grid, kThreads, st, src, rp, delta_out, delta_row_stride, x, gamma)
  DSQ_SWITCH_SRC(srck, DSQ_RS)
#undef DSQ_RS
  count_launches(1);
  return cudaGetLastError();
}

// Dense decode of a server payload and update of x.
__global__ void __launch_bounds__(kThreads) k_apply_dense(const PayloadView pv, float* x, uint64_t d, float gamma) {
  pdl_prologue();
  const uint64_t nq = (d + 3) / 4;
  for (uint64_t qd = (uint64_t)blockIdx.x * kThreads + threadIdx.x; qd < nq; qd += (uint64_t)gridDim.x * kThreads) {
    const uint64_t e = qd * 4;
    const uint32_t cnt = (uint32_t)min((uint64_t)4, d - e);
    float4 C;
    if (pv.op == DS_Q_IDENTITY) {
      C = load_row4(reinterpret_cast<const float*>(pv.base + pv.off[0]), e, cnt, 1);
    } else if (pv.op == DS_Q_SIGN1) {
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pv.base + pv.off[0]) + (e >> 5)) >> (uint32_t)(e & 31);
      const float s = __ldg(reinterpret_cast<const float*>(pv.base + pv.off[1]) + (e >> pv.log2_chunk));
      C = make_float4(signed_by_bit(s, w, 0), signed_by_bit(s, w, 1), signed_by_bit(s, w, 2), signed_by_bit(s, w, 3));
    } else if (pv.op == DS_Q_TERNARY) {
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pv.base + pv.off[0]) + (e >> 5)) >> (uint32_t)(e & 31);
      const uint32_t z = __ldg(reinterpret_cast<const uint32_t*>(pv.base + pv.off[1]) + (e >> 5)) >> (uint32_t)(e & 31);
      const float s = __ldg(reinterpret_cast<const float*>(pv.base + pv.off[2]));
      C = make_float4((z & 1u) ? signed_by_bit(s, w, 0) : 0.f, (z & 2u) ? signed_by_bit(s, w, 1) : 0.f,
                      (z & 4u) ? signed_by_bit(s, w, 2) : 0.f, (z & 8u) ? signed_by_bit(s, w, 3) : 0.f);
    } else if (pv.op == DS_Q_RSPARSE) {
      const uint32_t o = __ldg(reinterpret_cast<const uint32_t*>(pv.base + pv.off[1]) + (e >> pv.log2_chunk));
      const float* val = reinterpret_cast<const float*>(pv.base + pv.off[0]);
      C = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((uint32_t)k < cnt && (((uint32_t)e + k) & ((1u << pv.log2_keep) - 1u)) == o) comp(C, k) = __ldg(val + ((e + k) >> pv.log2_keep));
    } else if (pv.op == DS_Q_CLIP) {
      uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((uint32_t)k < cnt)
          w[k] = pv.clip_bits == 16 ? (uint32_t)__ldcs(reinterpret_cast<const uint16_t*>(pv.base + pv.off[0]) + e + k) << 16
                                    : (uint32_t)__ldcs(pv.base + pv.off[0] + e + k) << 24;
      C = make_float4(__uint_as_float(w[0]), __uint_as_float(w[1]), __uint_as_float(w[2]), __uint_as_float(w[3]));
    } else {  // DS_Q_QSGD
      const uint32_t lv = __ldcs(reinterpret_cast<const uint32_t*>(pv.base + pv.off[0] + e));
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pv.base + pv.off[1]) + (e >> 5)) >> (uint32_t)(e & 31);
      const float q = __ldg(reinterpret_cast<const float*>(pv.base + pv.off[2]) + (e >> pv.log2_chunk));
      C = make_float4(signed_by_bit(__fmul_rn(byte_to_float(lv, 0), q), w, 0),
                      signed_by_bit(__fmul_rn(byte_to_float(lv, 1), q), w, 1),
                      signed_by_bit(__fmul_rn(byte_to_float(lv, 2), q), w, 2),
                      signed_by_bit(__fmul_rn(byte_to_float(lv, 3), q), w, 3));
    }
    float4 xv = load_row4(x, e, cnt, 1);
    xv.x = __fsub_rn(xv.x, __fmul_rn(gamma, C.x)); xv.y = __fsub_rn(xv.y, __fmul_rn(gamma, C.y));
    xv.z = __fsub_rn(xv.z, __fmul_rn(gamma, C.z)); xv.w = __fsub_rn(xv.w, __fmul_rn(gamma, C.w));
    store_row4(x, e, cnt, 1, xv);
  }
}

// Sparse payload: only the k listed entries of x change (the others would subtract gamma * 0).
__global__ void __launch_bounds__(kThreads) k_apply_sparse(const uint32_t* __restrict__ idx, const float* __restrict__ val,
                                                           uint64_t k, float* x, float gamma) {
  pdl_prologue();
  for (uint64_t m = (uint64_t)blockIdx.x * kThreads + threadIdx.x; m < k; m += (uint64_t)gridDim.x * kThreads) {
    const uint32_t j = idx[m];
    x[j] = __fsub_rn(x[j], __fmul_rn(gamma, val[m]));
  }
}

cudaError_t launch_apply(const PayloadView& pv, float* x, uint64_t d, float gamma, cudaStream_t st) {
  if (pv.op == DS_Q_TOPK) {
    if (pv.k == 0) return cudaSuccess;
    launch_pdl(k_apply_sparse, grid_for(pv.k), kThreads, st, reinterpret_cast<const uint32_t*>(pv.base + pv.off[0]),
                                                        reinterpret_cast<const float*>(pv.base + pv.off[1]), pv.k, x, gamma);
  } else {
    launch_pdl(k_apply_dense, grid_for((d + 3) / 4), kThreads, st, pv, x, d, gamma);
  }
  count_launches(1);
  return cudaGetLastError();
}

// Sum of the n sparse worker payloads into the dense accumulator, workers added in order
// 0..n-1 as Eq. 4 is evaluated.
//
// k_sparse_offsets: for every worker, where each span of kAccSpan indices begins in its ascending
// index list (off[i][s] = first m with idx[m] >= s * kAccSpan; off[i][nspan] = k).
// k_sparse_accumulate: a CTA owns one span and builds its slice of the sum in shared memory: the
// entries of eight workers are fetched at once, then added worker by worker with a barrier in
// between (indices inside one payload are distinct, so one worker's additions never collide), and
// the finished slice is written out whole -- the accumulator needs no clearing beforehand.
constexpr uint32_t kAccSpan = kSparseSpan;

__global__ void __launch_bounds__(kThreads) k_sparse_offsets(const uint8_t* __restrict__ wp, uint64_t stride, uint64_t off_idx,
                                                             uint64_t k, uint64_t nspan, uint32_t* off) {
  pdl_prologue();
  const uint32_t i = blockIdx.y;
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(wp + (uint64_t)i * stride + off_idx);
  uint32_t* o = off + (uint64_t)i * (nspan + 1);
  for (uint64_t m = (uint64_t)blockIdx.x * kThreads + threadIdx.x; m <= k; m += (uint64_t)gridDim.x * kThreads) {
    // entry m opens every span after the one entry m-1 lies in, up to and including its own
    const uint64_t first = m == 0 ? 0 : (uint64_t)(idx[m - 1] / kAccSpan) + 1;
    uint64_t last = m == k ? nspan : (uint64_t)(idx[m] / kAccSpan);
    if (last > nspan) last = nspan;  // an index beyond d in a foreign payload must not leave the table
    for (uint64_t s = first; s <= last; ++s) o[s] = (uint32_t)m;
  }
}

__global__ void __launch_bounds__(kThreads) k_sparse_accumulate(const uint8_t* __restrict__ wp, uint64_t stride,
                                                                uint64_t off_idx, uint64_t off_val, uint32_t n, uint64_t d,
                                                                uint64_t nspan, const uint32_t* __restrict__ off,
                                                                float* acc) {
  pdl_prologue();
  __shared__ float s_acc[kAccSpan];
  const uint32_t tid = threadIdx.x;
  const uint64_t span = blockIdx.x;
  const uint32_t base = (uint32_t)(span * kAccSpan);
  for (uint32_t j = tid; j < kAccSpan; j += kThreads) s_acc[j] = 0.f;
  __syncthreads();
  for (uint32_t i0 = 0; i0 < n; i0 += 8) {
    // first entry of this thread in each of eight workers' slices, fetched before any is used
    uint32_t lo[8], hi[8], ji[8];
    float vi[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      lo[u] = 0; hi[u] = 0; ji[u] = 0; vi[u] = 0.f;
      if (i0 + u < n) {
        const uint32_t* o = off + (uint64_t)(i0 + u) * (nspan + 1) + span;
        lo[u] = o[0];
        hi[u] = o[1];
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (lo[u] + tid < hi[u]) {
        const uint8_t* pl = wp + (uint64_t)(i0 + u) * stride;
        ji[u] = reinterpret_cast<const uint32_t*>(pl + off_idx)[lo[u] + tid];
        vi[u] = reinterpret_cast<const float*>(pl + off_val)[lo[u] + tid];
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (i0 + u < n) {
        if (lo[u] + tid < hi[u]) {
          const uint32_t j = (ji[u] - base) & (kAccSpan - 1u);  // masked: never leaves the slice
          s_acc[j] = __fadd_rn(s_acc[j], vi[u]);
        }
        // a slice with more entries than threads (dense payloads) finishes here
        const uint8_t* pl = wp + (uint64_t)(i0 + u) * stride;
        for (uint32_t m = lo[u] + tid + kThreads; m < hi[u]; m += kThreads) {
          const uint32_t j = (reinterpret_cast<const uint32_t*>(pl + off_idx)[m] - base) & (kAccSpan - 1u);
          s_acc[j] = __fadd_rn(s_acc[j], reinterpret_cast<const float*>(pl + off_val)[m]);
        }
        __syncthreads();  // the next worker may add to the same entries
      }
    }
  }
  for (uint32_t j = tid * 4; j < kAccSpan; j += kThreads * 4) {
    const uint64_t e = (uint64_t)base + j;
    if (e + 4 <= d) {
      *reinterpret_cast<float4*>(acc + e) = make_float4(s_acc[j], s_acc[j + 1], s_acc[j + 2], s_acc[j + 3]);
    } else {
      for (uint32_t q = 0; q < 4; ++q)
        if (e + q < d) acc[e + q] = s_acc[j + q];
    }
  }
}

uint64_t sparse_offsets_bytes(uint32_t n, uint64_t d) { return (uint64_t)n * ((d + kAccSpan - 1) / kAccSpan + 1) * 4; }

cudaError_t launch_sparse_accumulate(const uint8_t* wp, uint64_t stride, uint64_t off_idx, uint64_t off_val, uint32_t n,
                                     uint64_t k, uint64_t d, uint32_t* offsets, bool offsets_ready, float* acc, cudaStream_t st) {
  const uint64_t nspan = (d + kAccSpan - 1) / kAccSpan;
  if (!offsets_ready) {
    uint64_t ctas = (k + kThreads) / kThreads;
    if (ctas > 148 * 8) ctas = 148 * 8;
    launch_pdl(k_sparse_offsets, dim3((unsigned)ctas, n, 1), kThreads, st, wp, stride, off_idx, k, nspan, offsets);
    count_launches(1);
  }
  launch_pdl(k_sparse_accumulate, (unsigned)nspan, kThreads, st, wp, stride, off_idx, off_val, n, d, nspan, offsets, acc);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace dsq
