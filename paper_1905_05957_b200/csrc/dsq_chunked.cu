// Chunk-wise operators fused with the error feedback: scaled 1-bit (Section 5.1 "1-bit
// compression") and randomised s-level quantisation (Section 3.2 "Randomized Quantization").
//
// One pass: load the pieces of v (Eq. 2 on the worker, Eq. 4 on the server), keep them in
// registers, reduce over the chunk, then emit payload, residual (Eq. 3 / Eq. 4) and, on a fused
// server pass, the model update.  v, Q[v] and delta never make a second trip through HBM.
//
// Geometry.  A chunk of L = 4*V*G entries is owned by G threads (G = 32..256, a power of two)
// that hold V float4 each; float4 number j of thread t covers entries (j*G + t)*4 .. +3 of the
// chunk, so a warp always touches 512 contiguous bytes.  A 256-thread CTA owns 256/G chunks.
//
// Reduction order.  The chunk sum is the pairwise sum in index order over the zero-padded chunk:
// two levels inside a float4, five xor-butterfly levels inside a warp (one 128-entry group), then
// a butterfly over the L/128 group sums through shared memory.  Float addition commutes bitwise,
// so every lane of a butterfly ends with the same value, independent of the launch shape.
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

template <int OP, int SRC, int V>
__global__ void __launch_bounds__(kThreads) k_chunked(const SrcParams src, const ChunkParams p) {
  __shared__ float s_red[64];
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t G = 1u << p.log2G;
  const uint32_t sub = tid >> p.log2G, t = tid & (G - 1u);
  const uint32_t row = blockIdx.y;
  const uint64_t c = (uint64_t)blockIdx.x * (kThreads >> p.log2G) + sub;  // chunk index in the row
  const uint32_t L = (uint32_t)V * G * 4u;
  const uint64_t d = src.d;
  const uint64_t base = c * L;
  const bool chunk_live = base < d;

  float4 v[V];
  uint32_t cnt[V];
#pragma unroll
  for (int j = 0; j < V; ++j) {
    const uint64_t e = base + (uint64_t)(j * G + t) * 4u;
    cnt[j] = e < d ? (uint32_t)min((uint64_t)4, d - e) : 0u;
    v[j] = cnt[j] ? src_load4<SRC>(src, row, e, cnt[j]) : make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // ---- chunk reduction: sum |v| (SIGN1) or sum v*v (QSGD), pairwise in index order
  const uint32_t NG = (V * G) >> 5;  // 128-entry groups per chunk
  float part[V];
#pragma unroll
  for (int j = 0; j < V; ++j) {
    float m0, m1, m2, m3;
    if constexpr (OP == DS_Q_SIGN1) {
      m0 = fabsf(v[j].x); m1 = fabsf(v[j].y); m2 = fabsf(v[j].z); m3 = fabsf(v[j].w);
    } else {
      m0 = __fmul_rn(v[j].x, v[j].x); m1 = __fmul_rn(v[j].y, v[j].y);
      m2 = __fmul_rn(v[j].z, v[j].z); m3 = __fmul_rn(v[j].w, v[j].w);
    }
    float s = __fadd_rn(__fadd_rn(m0, m1), __fadd_rn(m2, m3));
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
    part[j] = s;
  }
  float total;
  if (NG == 1) {
    total = part[0];
  } else {
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < V; ++j) s_red[sub * NG + j * (G >> 5) + (t >> 5)] = part[j];
    }
    __syncthreads();
    float x;
    if (NG <= 32) {
      x = lane < NG ? s_red[sub * NG + lane] : 0.f;
      for (uint32_t o = 1; o < NG; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
    } else {  // NG == 64
      x = __fadd_rn(s_red[sub * 64 + 2 * lane], s_red[sub * 64 + 2 * lane + 1]);
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
    }
    total = __shfl_sync(0xffffffffu, x, 0);
  }

  // ---- per-chunk quantities
  const uint32_t len = chunk_live ? (uint32_t)min((uint64_t)L, d - base) : 1u;
  float s_or_q, inv_q = 0.f;
  if constexpr (OP == DS_Q_SIGN1) {
    s_or_q = __fdiv_rn(total, (float)len);  // mean |v| over the true chunk length
    if (chunk_live && t == 0) p.out_scale[(uint64_t)row * p.scale_stride + c] = s_or_q;
  } else {
    float N = __fsqrt_rn(total);
    float q = 0.f;
    bool live = (N > 0.f) && (N < __int_as_float(0x7f800000));
    if (live) {
      inv_q = __fdiv_rn(p.levels_f, N);
      q = __fdiv_rn(N, p.levels_f);
      live = inv_q < __int_as_float(0x7f800000);
    }
    if (!live) { N = 0.f; q = 0.f; inv_q = 0.f; }
    s_or_q = q;
    if (chunk_live && t == 0) p.out_scale[(uint64_t)row * p.scale_stride + c] = N;
  }

  // ---- encode, residual, optional model update
  float* delta_row = p.delta_out + (uint64_t)row * p.delta_row_stride;
#pragma unroll
  for (int j = 0; j < V; ++j) {
    const uint32_t tq = (uint32_t)(j * G + t);  // float4 index inside the chunk
    const uint64_t e = base + (uint64_t)tq * 4u;
    float4 C;
    uint32_t nib = 0;
    if constexpr (OP == DS_Q_SIGN1) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const bool nonneg = compc(v[j], k) >= 0.f;
        nib |= (nonneg ? 1u : 0u) << k;
        comp(C, k) = nonneg ? s_or_q : -s_or_q;
      }
    } else {
      const uint4 rnd = philox4x32_10(make_uint4(tq, (uint32_t)c, p.server_pass ? 0xFFFFFFFFu : row, p.step),
                                      p.key0, p.key1);
      const uint32_t w[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
      uint32_t packed = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float val = compc(v[j], k);
        const float u = __fmul_rn(__uint2float_rn(w[k] >> 8), 5.9604644775390625e-08f);  // 2^-24, exact
        float r = __fmul_rn(fabsf(val), inv_q);
        r = fminf(r, p.levels_f);
        const float f = floorf(r);
        const float pr = __fsub_rn(r, f);
        uint32_t level = (uint32_t)f + (u < pr ? 1u : 0u);
        level = min(level, p.levels_u);
        const float mag = __fmul_rn((float)level, s_or_q);
        const bool nonneg = val >= 0.f;
        nib |= (nonneg ? 1u : 0u) << k;
        comp(C, k) = nonneg ? mag : -mag;
        packed |= level << (8 * k);
      }
      if (cnt[j]) *reinterpret_cast<uint32_t*>(p.out_lvl + (uint64_t)row * p.lvl_stride + e) = packed;
    }
    // sign words: eight neighbouring lanes hold one 32-entry word
    nib &= (1u << cnt[j]) - 1u;
    uint32_t word = nib << ((lane & 7u) * 4u);
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    word |= __shfl_xor_sync(0xffffffffu, word, 4);
    if ((lane & 7u) == 0 && cnt[j]) p.out_bits[(uint64_t)row * p.bits_stride + (e >> 5)] = word;

    if (cnt[j]) {
      float4 dl;
      dl.x = __fsub_rn(v[j].x, C.x); dl.y = __fsub_rn(v[j].y, C.y);
      dl.z = __fsub_rn(v[j].z, C.z); dl.w = __fsub_rn(v[j].w, C.w);
      store_row4(delta_row, e, cnt[j], src.vec, dl);
      if (p.x) {  // fused model update (server pass only): x = x - gamma * Q[v]
        float4 xv = load_row4(p.x, e, cnt[j], 1);
        xv.x = __fsub_rn(xv.x, __fmul_rn(p.gamma, C.x)); xv.y = __fsub_rn(xv.y, __fmul_rn(p.gamma, C.y));
        xv.z = __fsub_rn(xv.z, __fmul_rn(p.gamma, C.z)); xv.w = __fsub_rn(xv.w, __fmul_rn(p.gamma, C.w));
        store_row4(p.x, e, cnt[j], 1, xv);
      }
    }
  }
}

template <int OP, int SRC>
static cudaError_t launch_v(const SrcParams& src, ChunkParams p, uint32_t rows, uint32_t chunk, cudaStream_t st) {
  // chunk = 4*V*G with G <= 256: V = 1 for chunk <= 1024, else chunk/1024
  const uint32_t V = chunk <= 1024 ? 1u : chunk / 1024u;
  const uint32_t G = chunk / (4u * V);
  uint32_t log2G = 0;
  while ((1u << log2G) < G) ++log2G;
  p.log2G = log2G;
  const uint64_t nc = (src.d + chunk - 1) / chunk;
  const uint32_t cpc = kThreads / G;
  dim3 grid((unsigned)((nc + cpc - 1) / cpc), rows, 1);
  switch (V) {
    case 1: k_chunked<OP, SRC, 1><<<grid, kThreads, 0, st>>>(src, p); break;
    case 2: k_chunked<OP, SRC, 2><<<grid, kThreads, 0, st>>>(src, p); break;
    case 4: k_chunked<OP, SRC, 4><<<grid, kThreads, 0, st>>>(src, p); break;
    case 8: k_chunked<OP, SRC, 8><<<grid, kThreads, 0, st>>>(src, p); break;
    default: return cudaErrorInvalidValue;
  }
  count_launches(1);
  return cudaGetLastError();
}

template <int OP>
static cudaError_t launch_src(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                              cudaStream_t st) {
  switch (srck) {
    case SRC_WORKER: return launch_v<OP, SRC_WORKER>(src, p, rows, chunk, st);
    case SRC_SRV_IDENTITY: return launch_v<OP, SRC_SRV_IDENTITY>(src, p, rows, chunk, st);
    case SRC_SRV_SIGN1: return launch_v<OP, SRC_SRV_SIGN1>(src, p, rows, chunk, st);
    case SRC_SRV_TOPK: return launch_v<OP, SRC_SRV_TOPK>(src, p, rows, chunk, st);
    case SRC_SRV_QSGD: return launch_v<OP, SRC_SRV_QSGD>(src, p, rows, chunk, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_chunked(int op, int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                           cudaStream_t st) {
  if (op == DS_Q_SIGN1) return launch_src<DS_Q_SIGN1>(srck, src, p, rows, chunk, st);
  if (op == DS_Q_QSGD) return launch_src<DS_Q_QSGD>(srck, src, p, rows, chunk, st);
  return cudaErrorInvalidValue;
}

}  // namespace dsq
