// Elementwise kernels: Q = identity (Algorithm 1 then is parallel SGD, Section 1), the stand-alone
// model update x = x - gamma Q[v] (Algorithm 1, last line of the loop), and the ordered
// accumulation of sparse worker payloads for the server mean (first line of Eq. 4).
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

template <int SRC>
__global__ void __launch_bounds__(kThreads) k_identity(const SrcParams src, float* out_c, uint64_t c_row_stride,
                                                       float* delta_out, uint64_t delta_row_stride, float* x,
                                                       float gamma) {
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
    store_row4(delta_out + (uint64_t)row * delta_row_stride, e, cnt, src.vec, make_float4(0.f, 0.f, 0.f, 0.f));
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
#define DSQ_ID(S) k_identity<S><<<grid, kThreads, 0, st>>>(src, out_c, c_row_stride, delta_out, delta_row_stride, x, gamma)
  switch (srck) {
    case SRC_WORKER: DSQ_ID(SRC_WORKER); break;
    case SRC_SRV_IDENTITY: DSQ_ID(SRC_SRV_IDENTITY); break;
    case SRC_SRV_SIGN1: DSQ_ID(SRC_SRV_SIGN1); break;
    case SRC_SRV_TOPK: DSQ_ID(SRC_SRV_TOPK); break;
    case SRC_SRV_QSGD: DSQ_ID(SRC_SRV_QSGD); break;
    default: return cudaErrorInvalidValue;
  }
#undef DSQ_ID
  count_launches(1);
  return cudaGetLastError();
}

// Dense decode of a server payload and update of x.
__global__ void __launch_bounds__(kThreads) k_apply_dense(const PayloadView pv, float* x, uint64_t d, float gamma) {
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
  for (uint64_t m = (uint64_t)blockIdx.x * kThreads + threadIdx.x; m < k; m += (uint64_t)gridDim.x * kThreads) {
    const uint32_t j = idx[m];
    x[j] = __fsub_rn(x[j], __fmul_rn(gamma, val[m]));
  }
}

cudaError_t launch_apply(const PayloadView& pv, float* x, uint64_t d, float gamma, cudaStream_t st) {
  if (pv.op == DS_Q_TOPK) {
    if (pv.k == 0) return cudaSuccess;
    k_apply_sparse<<<grid_for(pv.k), kThreads, 0, st>>>(reinterpret_cast<const uint32_t*>(pv.base + pv.off[0]),
                                                        reinterpret_cast<const float*>(pv.base + pv.off[1]), pv.k, x, gamma);
  } else {
    k_apply_dense<<<grid_for((d + 3) / 4), kThreads, 0, st>>>(pv, x, d, gamma);
  }
  count_launches(1);
  return cudaGetLastError();
}

// Sum of the n sparse worker payloads into the dense accumulator, workers added in order
// 0..n-1 as Eq. 4 is evaluated.  A CTA owns a span of indices: it first finds, for up to 128
// workers at a time, where that span begins and ends in each worker's ascending index list
// (binary searches, all in parallel), then walks the workers in order with a barrier in between.
// Indices inside one payload are distinct, so the additions of one worker never collide, and no
// other CTA touches this span.
constexpr uint32_t kAccSpan = 8192;

__global__ void __launch_bounds__(kThreads) k_sparse_accumulate_all(const uint8_t* __restrict__ wp, uint64_t stride,
                                                                    uint64_t off_idx, uint64_t off_val, uint32_t n,
                                                                    uint64_t k, uint64_t d, float* acc) {
  __shared__ uint64_t s_bound[2 * 128];
  const uint32_t tid = threadIdx.x;
  const uint64_t span_lo = (uint64_t)blockIdx.x * kAccSpan;
  const uint64_t span_hi = min(span_lo + kAccSpan, d);
  for (uint32_t i0 = 0; i0 < n; i0 += 128) {
    const uint32_t nb = min(128u, n - i0);
    if (tid < 2 * nb) {
      const uint32_t* idx = reinterpret_cast<const uint32_t*>(wp + (uint64_t)(i0 + (tid >> 1)) * stride + off_idx);
      const uint64_t bound = (tid & 1u) ? span_hi : span_lo;
      uint64_t lo = 0, hi = k;  // first m with idx[m] >= bound
      while (lo < hi) {
        const uint64_t mid = (lo + hi) >> 1;
        if (idx[mid] < bound) lo = mid + 1; else hi = mid;
      }
      s_bound[tid] = lo;
    }
    __syncthreads();
    for (uint32_t u = 0; u < nb; ++u) {
      const uint8_t* pl = wp + (uint64_t)(i0 + u) * stride;
      const uint32_t* idx = reinterpret_cast<const uint32_t*>(pl + off_idx);
      const float* val = reinterpret_cast<const float*>(pl + off_val);
      const uint64_t hi = s_bound[2 * u + 1];
      for (uint64_t m = s_bound[2 * u] + tid; m < hi; m += kThreads) {
        const uint32_t j = idx[m];
        acc[j] = __fadd_rn(acc[j], val[m]);
      }
      __syncthreads();  // the next worker may add to the same entries
    }
  }
}

cudaError_t launch_sparse_accumulate(const uint8_t* wp, uint64_t stride, uint64_t off_idx, uint64_t off_val, uint32_t n,
                                     uint64_t k, uint64_t d, float* acc, cudaStream_t st) {
  if (k == 0 || n == 0) return cudaSuccess;
  k_sparse_accumulate_all<<<(unsigned)((d + kAccSpan - 1) / kAccSpan), kThreads, 0, st>>>(wp, stride, off_idx, off_val, n, k,
                                                                                          d, acc);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace dsq
