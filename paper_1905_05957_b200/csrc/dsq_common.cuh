// Shared device-side pieces of the DoubleSqueeze kernels: parameter blocks, the "source" of the
// vector that is about to be compressed (worker: g + delta, Eq. 2; server: decoded mean of the
// worker payloads + delta, Eq. 4), and the Philox4x32-10 generator.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsq {

constexpr int kThreads = 256;  // every streaming kernel uses 256-thread CTAs

enum Src : int {
  SRC_WORKER = 0,        // v = g[row] + delta_w[row]
  SRC_SRV_IDENTITY = 1,  // v = (sum_i c_i) * inv_n + delta_s
  SRC_SRV_SIGN1 = 2,
  SRC_SRV_TOPK = 3,      // the sparse payloads were summed into a dense accumulator beforehand
  SRC_SRV_QSGD = 4,
};

// Where v comes from.  Worker payload sub-arrays follow the documented payload layout.
struct SrcParams {
  const float* g;          // worker: gradients [n, d]
  const float* delta;      // worker: delta_w [n, d]; server: delta_s [d]
  uint64_t d;
  uint32_t n;              // server: number of payloads to average
  float inv_n;             // server: 1/n rounded once
  const uint8_t* wp;       // server: base of the n worker payloads
  uint64_t wp_stride;      // bytes between payloads
  uint64_t wp_off[3];      // sub-array offsets inside a payload
  uint32_t w_log2_chunk;   // worker chunk length (SIGN1, QSGD)
  float w_levels;          // worker QSGD level count as a float
  float* acc;              // SRC_SRV_TOPK: dense accumulator [d]; cleared as it is consumed
  int vec;                 // 1 if every row starts 16-byte aligned (d % 4 == 0)
};

__device__ __forceinline__ float4 ld_stream4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st_stream4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

__device__ __forceinline__ float& comp(float4& v, int k) { return (&v.x)[k]; }
__device__ __forceinline__ float compc(const float4& v, int k) { return (&v.x)[k]; }

// Loads the four entries e..e+3 of a length-d row starting at `base`; entries >= cnt read as +0.
__device__ __forceinline__ float4 load_row4(const float* base, uint64_t e, uint32_t cnt, int vec) {
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  if (vec && cnt == 4) {
    r = ld_stream4(base + e);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((uint32_t)k < cnt) comp(r, k) = __ldcs(base + e + k);
  }
  return r;
}

__device__ __forceinline__ void store_row4(float* base, uint64_t e, uint32_t cnt, int vec, float4 v) {
  if (vec && cnt == 4) {
    st_stream4(base + e, v);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((uint32_t)k < cnt) __stcs(base + e + k, compc(v, k));
  }
}

// The vector to compress, four consecutive entries at offset e of row `row`.  cnt in [1, 4] is the
// number of entries that exist (e + cnt <= d); the others are returned as +0.
template <int SRC>
__device__ __forceinline__ float4 src_load4(const SrcParams& p, uint32_t row, uint64_t e, uint32_t cnt) {
  if constexpr (SRC == SRC_WORKER) {
    const uint64_t off = (uint64_t)row * p.d;
    float4 a = load_row4(p.g + off, e, cnt, p.vec);
    float4 b = load_row4(p.delta + off, e, cnt, p.vec);
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
  } else {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if constexpr (SRC == SRC_SRV_IDENTITY) {
      for (uint32_t i = 0; i < p.n; ++i) {
        const float* c = reinterpret_cast<const float*>(p.wp + i * p.wp_stride + p.wp_off[0]);
        float4 ci = load_row4(c, e, cnt, 1);
        acc.x = __fadd_rn(acc.x, ci.x); acc.y = __fadd_rn(acc.y, ci.y);
        acc.z = __fadd_rn(acc.z, ci.z); acc.w = __fadd_rn(acc.w, ci.w);
      }
    } else if constexpr (SRC == SRC_SRV_SIGN1) {
      const uint64_t word = e >> 5;
      const uint32_t sh = (uint32_t)(e & 31);
      const uint64_t ch = e >> p.w_log2_chunk;
      for (uint32_t i = 0; i < p.n; ++i) {
        const uint8_t* pl = p.wp + i * p.wp_stride;
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pl + p.wp_off[0]) + word) >> sh;
        const float s = __ldg(reinterpret_cast<const float*>(pl + p.wp_off[1]) + ch);
        acc.x = __fadd_rn(acc.x, (w & 1u) ? s : -s); acc.y = __fadd_rn(acc.y, (w & 2u) ? s : -s);
        acc.z = __fadd_rn(acc.z, (w & 4u) ? s : -s); acc.w = __fadd_rn(acc.w, (w & 8u) ? s : -s);
      }
    } else if constexpr (SRC == SRC_SRV_QSGD) {
      const uint64_t word = e >> 5;
      const uint32_t sh = (uint32_t)(e & 31);
      const uint64_t ch = e >> p.w_log2_chunk;
      for (uint32_t i = 0; i < p.n; ++i) {
        const uint8_t* pl = p.wp + i * p.wp_stride;
        const uint32_t lv = __ldcs(reinterpret_cast<const uint32_t*>(pl + p.wp_off[0] + e));
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pl + p.wp_off[1]) + word) >> sh;
        const float nrm = __ldg(reinterpret_cast<const float*>(pl + p.wp_off[2]) + ch);
        const float q = __fdiv_rn(nrm, p.w_levels);
        const float m0 = __fmul_rn((float)(lv & 255u), q), m1 = __fmul_rn((float)((lv >> 8) & 255u), q);
        const float m2 = __fmul_rn((float)((lv >> 16) & 255u), q), m3 = __fmul_rn((float)(lv >> 24), q);
        acc.x = __fadd_rn(acc.x, (w & 1u) ? m0 : -m0); acc.y = __fadd_rn(acc.y, (w & 2u) ? m1 : -m1);
        acc.z = __fadd_rn(acc.z, (w & 4u) ? m2 : -m2); acc.w = __fadd_rn(acc.w, (w & 8u) ? m3 : -m3);
      }
    } else {  // SRC_SRV_TOPK
      acc = load_row4(p.acc, e, cnt, p.vec);
      store_row4(p.acc, e, cnt, p.vec, make_float4(0.f, 0.f, 0.f, 0.f));
    }
    float4 ds = load_row4(p.delta, e, cnt, p.vec);
    float4 v;
    v.x = __fadd_rn(__fmul_rn(acc.x, p.inv_n), ds.x); v.y = __fadd_rn(__fmul_rn(acc.y, p.inv_n), ds.y);
    v.z = __fadd_rn(__fmul_rn(acc.z, p.inv_n), ds.z); v.w = __fadd_rn(__fmul_rn(acc.w, p.inv_n), ds.w);
    // entries past the end must read as +0 whatever the payload padding holds
    if (cnt < 4) {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((uint32_t)k >= cnt) comp(v, k) = 0.f;
    }
    return v;
  }
}

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors, the key
// advanced by the two Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

}  // namespace dsq
