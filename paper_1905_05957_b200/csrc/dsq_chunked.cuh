// Chunk-wise operators fused with the error feedback: scaled 1-bit (Section 5.1 "1-bit
// compression") and randomised s-level quantisation (Section 3.2 "Randomized Quantization").
//
// One pass: load the pieces of v (Eq. 2 on the worker, Eq. 4 on the server), keep them in
// registers, reduce over the chunk, then emit payload, residual (Eq. 3 / Eq. 4) and, on a fused
// server pass, the model update.  v, Q[v] and delta never make a second trip through HBM.
//
// Geometry.  A chunk of L = 4*V*G entries is owned by G threads (G = 32..256, a power of two)
// that hold V float4 each; float4 number j ("row" j) of thread t covers entries (j*G + t)*4 .. +3
// of the chunk, so a warp always touches 512 contiguous bytes.  A 256-thread CTA owns 256/G chunks.
//
// Reduction order.  The chunk sum is the pairwise sum in index order over the zero-padded chunk:
// two levels inside a float4, five xor-butterfly levels inside a warp (one 128-entry group), then
// a butterfly over the L/128 group sums through shared memory.  Float addition commutes bitwise,
// so the value does not depend on which lane performs an addition.  The V butterflies of a warp
// are folded into one: at level s a lane keeps the rows whose bit s equals its own lane bit s and
// hands the others to its partner, so that V rows cost log2(V) halving steps plus 5 - log2(V)
// ordinary ones instead of 5 V shuffles, with the same additions in the same tree.
#pragma once
#include "dsq_common.cuh"
#include "dsq_internal.h"

namespace dsq {

namespace {

// Template code of the 1-bit operator whose scale comes from l2 magnitudes (DS_NORM_L2); the
// other values of OP are the ds_op codes.
constexpr int kOpSign1L2 = 101;
// ... and of the quantiser run over a window of the problem (some of the workers, or a slice of d):
// its Philox counters carry the offsets of the window.  A separate instantiation, so that the
// whole-vector kernels stay exactly as they were (the two extra additions cost them registers).
constexpr int kOpQsgdWindow = 103;

// Sum over the warp of row (lane % V) of a[.]; the butterfly order is lane bit 0, 1, ..., 4.
template <int V>
__device__ __forceinline__ float warp_rows_sum(float (&a)[V], uint32_t lane) {
  int s = 0;
#pragma unroll
  for (int n = V; n > 1; n >>= 1, ++s) {
    const bool up = (lane >> s) & 1u;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float keep = up ? a[2 * i + 1] : a[2 * i];
      const float send = up ? a[2 * i] : a[2 * i + 1];
      a[i] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, 1 << s));
    }
  }
  float x = a[0];
#pragma unroll
  for (int o = V; o < 32; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

// Each lane holds one 4-bit field per row (signs of its float4).  Returns the 32-entry sign word
// of row (lane % V) for the eight lanes lane&~7 .. lane|7 (valid in every lane of the octet whose
// lane % V names that row).  Same halving idea: log2(V) exchange steps, then OR-combining steps.
template <int V>
__device__ __forceinline__ uint32_t octet_sign_words(const uint32_t (&nib)[V], uint32_t lane) {
  uint32_t f[V];
#pragma unroll
  for (int r = 0; r < V; ++r) f[r] = nib[r];
  int s = 0;
  int w = 4;  // field width in bits
#pragma unroll
  for (int n = V; n > 1; n >>= 1, ++s, w <<= 1) {
    const bool up = (lane >> s) & 1u;
    uint32_t send = 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) send |= (up ? f[2 * i] : f[2 * i + 1]) << (i * w);
    const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1 << s);
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const uint32_t keep = up ? f[2 * i + 1] : f[2 * i];
      const uint32_t got = (recv >> (i * w)) & ((1u << w) - 1u);  // w <= 16 inside this loop
      f[i] = up ? (got | (keep << w)) : (keep | (got << w));      // the lower lane's entries come first
    }
  }
  uint32_t x = f[0];
#pragma unroll
  for (int o = V; o < 8; o <<= 1, w <<= 1) {
    const bool up = (lane & o) != 0;
    const uint32_t got = __shfl_xor_sync(0xffffffffu, x, o);
    x = up ? (got | (x << w)) : (x | (got << w));
  }
  return x;
}

// Pairwise sum over a chunk: part[j] is the calling thread's sum over its float4 number j (entries
// (j*G + t)*4 .. +3 of the chunk, already added as (a+b)+(c+d)).  Every thread of the chunk returns the
// chunk total.  Called by all threads of the CTA (one barrier when the chunk spans several warps).
template <int V, int LOG2G>
__device__ __forceinline__ float chunk_total(float (&part)[V], float* s_red) {
  constexpr uint32_t G = 1u << LOG2G;
  constexpr uint32_t NG = (V * G) >> 5;   // 128-entry groups per chunk
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t sub = tid >> LOG2G, t = tid & (G - 1u);
  float total = warp_rows_sum<V>(part, lane);  // lane holds the 128-entry group sum of row lane % V
  if constexpr (NG > 1) {
    // group index inside the chunk: row j = lane, warp (t >> 5) of the row
    if (lane < (uint32_t)V) s_red[sub * NG + lane * (G >> 5) + (t >> 5)] = total;
    __syncthreads();
    float x;
    if constexpr (NG <= 32) {
      x = lane < NG ? s_red[sub * NG + lane] : 0.f;
#pragma unroll
      for (uint32_t o = 1; o < NG; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
    } else {  // NG == 64
      x = __fadd_rn(s_red[sub * 64 + 2 * lane], s_red[sub * 64 + 2 * lane + 1]);
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
    }
    total = __shfl_sync(0xffffffffu, x, 0);
  }
  return total;
}

template <int OP, int SRC, int V, int LOG2G, bool FULL>
__device__ __forceinline__ void chunk_body(const SrcParams& src, const ChunkParams& p, float* s_red, float* s_scal) {
  constexpr uint32_t G = 1u << LOG2G;
  constexpr uint32_t L = (uint32_t)V * G * 4u;
  constexpr uint32_t CPC = kThreads / G;  // chunks per CTA
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t sub = tid >> LOG2G, t = tid & (G - 1u);
  const uint32_t row = blockIdx.y;
  const uint64_t c = (uint64_t)blockIdx.x * CPC + sub;  // chunk index in the row
  const uint64_t d = src.d;
  const uint64_t base = c * L;
  const bool chunk_live = FULL || base < d;

  float4 v[V];
  uint32_t cnt[V];
  if constexpr (FULL && SRC == SRC_WORKER) {
    const float4* gp = reinterpret_cast<const float4*>(src.g + (uint64_t)row * d + base) + t;
    const float4* dp = reinterpret_cast<const float4*>(src.delta + (uint64_t)row * d + base) + t;
    float4 a[V], b[V];
#pragma unroll
    for (int j = 0; j < V; ++j) a[j] = __ldcs(gp + j * G);
#pragma unroll
    for (int j = 0; j < V; ++j) b[j] = __ldcs(dp + j * G);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      cnt[j] = 4;
      v[j] = add4_rn(a[j], b[j]);
    }
  } else {
    uint64_t e[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
      e[j] = base + (uint64_t)(j * G + t) * 4u;
      cnt[j] = FULL ? 4u : (e[j] < d ? (uint32_t)min((uint64_t)4, d - e[j]) : 0u);
    }
    src_load_tile<SRC, V>(src, row, e, cnt, v);
  }

  // fused model update (server pass): fetch x now so that its latency hides behind the reduction
  constexpr bool kServer = !is_worker_src(SRC);  // only a server pass can carry the update
  float4 xv[kServer ? V : 1];
  if (kServer && p.x) {
#pragma unroll
    for (int j = 0; j < V; ++j)
      xv[kServer ? j : 0] = cnt[j] ? load_row4(p.x, base + (uint64_t)(j * G + t) * 4u, cnt[j], 1) : make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // ---- chunk reduction: sum |v| (SIGN1) or sum v*v (SIGN1 with l2 magnitudes, QSGD), pairwise in index order
  float part[V];
#pragma unroll
  for (int j = 0; j < V; ++j) {
    float m0, m1, m2, m3;
    if constexpr (OP == DS_Q_SIGN1) {
      m0 = fabsf(v[j].x); m1 = fabsf(v[j].y); m2 = fabsf(v[j].z); m3 = fabsf(v[j].w);
    } else {
      const float4 sq = mul4_rn(v[j], v[j]);
      m0 = sq.x; m1 = sq.y; m2 = sq.z; m3 = sq.w;
    }
    part[j] = __fadd_rn(__fadd_rn(m0, m1), __fadd_rn(m2, m3));
  }
  const float total = chunk_total<V, LOG2G>(part, s_red);

  // ---- per-chunk quantities
  const uint32_t len = FULL ? L : (chunk_live ? (uint32_t)min((uint64_t)L, d - base) : 1u);
  float s_or_q, inv_q = 0.f;
  if constexpr (OP == DS_Q_SIGN1 || OP == kOpSign1L2) {
    // ratio of the magnitudes of v_c and sign(v_c) over the true chunk length: mean |v|, or with
    // l2 magnitudes ||v_c||_2 / sqrt(len)
    s_or_q = OP == kOpSign1L2 ? __fdiv_rn(__fsqrt_rn(total), __fsqrt_rn((float)len)) : __fdiv_rn(total, (float)len);
    if (chunk_live && t == 0) p.out_scale[(uint64_t)row * p.scale_stride + c] = s_or_q;
  } else {
    // square root and the two divisions once per chunk (its first warp), not once per thread
    float q = 0.f;
    if (G == 32 || (t >> 5) == 0) {
      float N = __fsqrt_rn(total);
      bool live = (N > 0.f) && (N < __int_as_float(0x7f800000));
      if (live) {
        inv_q = __fdiv_rn(p.levels_f, N);
        q = __fdiv_rn(N, p.levels_f);
        live = inv_q < __int_as_float(0x7f800000);
      }
      if (!live) { q = 0.f; inv_q = 0.f; }
      if (G > 32 && lane == 0) { s_scal[2 * sub] = q; s_scal[2 * sub + 1] = inv_q; }
    }
    if constexpr (G > 32) {
      __syncthreads();
      q = s_scal[2 * sub];
      inv_q = s_scal[2 * sub + 1];
    }
    s_or_q = q;
    if (chunk_live && t == 0) p.out_scale[(uint64_t)row * p.scale_stride + c] = q;  // the grid step is what is sent
  }

  // ---- encode, residual, optional model update
  float* delta_chunk = p.delta_out + (uint64_t)row * p.delta_row_stride + base;
  uint32_t nib[V];
#pragma unroll
  for (int j = 0; j < V; ++j) {
    const uint32_t tq = (uint32_t)(j * G + t);  // float4 index inside the chunk
    const uint64_t e = base + (uint64_t)tq * 4u;
    float4 C;
    nib[j] = 0;
    if constexpr (OP == DS_Q_SIGN1 || OP == kOpSign1L2) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const bool nonneg = compc(v[j], k) >= 0.f;
        nib[j] |= (nonneg ? 1u : 0u) << k;
        comp(C, k) = nonneg ? s_or_q : -s_or_q;
      }
    } else {
      const uint4 rnd = philox4x32_10(make_uint4(tq, OP == kOpQsgdWindow ? (uint32_t)c + p.chunk0 : (uint32_t)c,
                                                  p.server_pass ? 0xFFFFFFFFu : (OP == kOpQsgdWindow ? row + p.row0 : row), p.step), p.keys);
      const uint32_t w[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
      uint32_t lb[4];
      // r = |v| * (s / N), clamped to s
      float4 r4 = mul4_rn(make_float4(fabsf(v[j].x), fabsf(v[j].y), fabsf(v[j].z), fabsf(v[j].w)),
                          make_float4(inv_q, inv_q, inv_q, inv_q));
      r4 = make_float4(fminf(r4.x, p.levels_f), fminf(r4.y, p.levels_f), fminf(r4.z, p.levels_f), fminf(r4.w, p.levels_f));
      // floor(r) for 0 <= r <= 255 without a conversion: adding 2^23 with rounding toward zero
      // leaves 2^23 + floor(r), whose low mantissa byte is the integer and whose difference
      // from 2^23 is the float
      float4 tz4, f4;
      {
        const f32x2 big = pack2(8388608.0f, 8388608.0f), nbig = pack2(-8388608.0f, -8388608.0f);
        const f32x2 t01 = add2_rz(pack2(r4.x, r4.y), big), t23 = add2_rz(pack2(r4.z, r4.w), big);
        unpack2(t01, tz4.x, tz4.y);
        unpack2(t23, tz4.z, tz4.w);
        unpack2(add2_rn(t01, nbig), f4.x, f4.y);
        unpack2(add2_rn(t23, nbig), f4.z, f4.w);
      }
      const float4 pr4 = sub4_rn(r4, f4);  // exact
      float4 lf4;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float u = __fmul_rn(__uint2float_rn(w[k] >> 8), 5.9604644775390625e-08f);  // 2^-24, exact
        const bool up = u < compc(pr4, k);
        lb[k] = __float_as_uint(compc(tz4, k)) + (up ? 1u : 0u);      // low byte = level (no carry: r = 255 has pr = 0)
        comp(lf4, k) = up ? __fadd_rn(compc(f4, k), 1.0f) : compc(f4, k);  // the level as a float, exact
      }
      const float4 mag4 = mul4_rn(lf4, make_float4(s_or_q, s_or_q, s_or_q, s_or_q));
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const bool nonneg = compc(v[j], k) >= 0.f;
        nib[j] |= (nonneg ? 1u : 0u) << k;
        comp(C, k) = nonneg ? compc(mag4, k) : -compc(mag4, k);
      }
      const uint32_t packed = __byte_perm(__byte_perm(lb[0], lb[1], 0x0040), __byte_perm(lb[2], lb[3], 0x0040), 0x5410);
      if (cnt[j]) *reinterpret_cast<uint32_t*>(p.out_lvl + (uint64_t)row * p.lvl_stride + e) = packed;
    }
    if constexpr (!FULL) nib[j] &= (1u << cnt[j]) - 1u;  // pad bits are 0

    if (cnt[j]) {
      // the residual (Eq. 3 / Eq. 4) -- unless no error is carried: a plain worker never keeps one, a
      // server pass without compensation has no destination for it
      if (SRC != SRC_WORKER_PLAIN && (SRC == SRC_WORKER || p.delta_out)) {
        const float4 dl = sub4_rn(v[j], C);
        if constexpr (FULL) {
          st_stream4(delta_chunk + tq * 4u, dl);
        } else {
          store_row4(delta_chunk, (uint64_t)tq * 4u, cnt[j], src.vec, dl);
        }
      }
      if (kServer && p.x) {  // fused model update (server pass only): x = x - gamma * Q[v]
        const float4 xo = xv[kServer ? j : 0];
        float4 xn;  // scalar: a multiply that feeds a subtract must not be contracted
        xn.x = __fsub_rn(xo.x, __fmul_rn(p.gamma, C.x)); xn.y = __fsub_rn(xo.y, __fmul_rn(p.gamma, C.y));
        xn.z = __fsub_rn(xo.z, __fmul_rn(p.gamma, C.z)); xn.w = __fsub_rn(xo.w, __fmul_rn(p.gamma, C.w));
        store_row4(p.x, e, cnt[j], 1, xn);
      }
    }
  }
  // sign words: eight neighbouring lanes hold one 32-entry word per row; lane (octet base + r)
  // stores the word of row r
  const uint32_t word = octet_sign_words<V>(nib, lane);
  const uint32_t r = lane & 7u;
  if (r < (uint32_t)V) {
    const uint64_t e0 = base + (uint64_t)(r * G + (t & ~7u)) * 4u;  // first entry of that word
    if (FULL || e0 < d) p.out_bits[(uint64_t)row * p.bits_stride + (e0 >> 5)] = word;
  }
}

// Resident CTAs the kernel is compiled for.  Worker passes take what the compiler gives, except the
// windowed quantiser: its worker pass is bound by instruction issue and wants six CTAs (40
// registers, what the whole-vector kernel gets by itself; with 48 it measured 8 % slower).  Server
// passes see kServerCtasPerSm.
constexpr int chunk_ctas(int op, int src, int v) {
  if (is_worker_src(src)) return (op == kOpQsgdWindow && v <= 2) ? 6 : 0;
  return v >= 8 ? 2 : kServerCtasPerSm;
}

template <int OP, int SRC, int V, int LOG2G>
__global__ void __launch_bounds__(kThreads, chunk_ctas(OP, SRC, V)) k_chunked(const SrcParams src, const ChunkParams p) {
  pdl_prologue();
  __shared__ float s_red[64];
  __shared__ float s_scal[16];
  constexpr uint64_t span = (uint64_t)V * 4u * kThreads;  // entries per CTA
  // interior CTA of an aligned row: no bounds logic anywhere
  if (src.vec && ((uint64_t)blockIdx.x + 1) * span <= src.d) {
    chunk_body<OP, SRC, V, LOG2G, true>(src, p, s_red, s_scal);
  } else {
    chunk_body<OP, SRC, V, LOG2G, false>(src, p, s_red, s_scal);
  }
}

template <int OP, int SRC>
cudaError_t launch_v(const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk, cudaStream_t st) {
  // chunk = 4*V*G with G <= 256: V = 1 for chunk <= 1024, else chunk/1024
  const uint64_t span_entries = chunk <= 1024 ? 1024 : chunk;  // entries per CTA
  dim3 grid((unsigned)((src.d + span_entries - 1) / span_entries), rows, 1);
  switch (chunk) {
    case 128: launch_pdl(k_chunked<OP, SRC, 1, 5>, grid, kThreads, st, src, p); break;
    case 256: launch_pdl(k_chunked<OP, SRC, 1, 6>, grid, kThreads, st, src, p); break;
    case 512: launch_pdl(k_chunked<OP, SRC, 1, 7>, grid, kThreads, st, src, p); break;
    case 1024: launch_pdl(k_chunked<OP, SRC, 1, 8>, grid, kThreads, st, src, p); break;
    case 2048: launch_pdl(k_chunked<OP, SRC, 2, 8>, grid, kThreads, st, src, p); break;
    case 4096: launch_pdl(k_chunked<OP, SRC, 4, 8>, grid, kThreads, st, src, p); break;
    case 8192: launch_pdl(k_chunked<OP, SRC, 8, 8>, grid, kThreads, st, src, p); break;
    default: return cudaErrorInvalidValue;
  }
  count_launches(1);
  return cudaGetLastError();
}

template <int OP>
cudaError_t launch_src(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                       cudaStream_t st) {
  switch (srck) {
    case SRC_WORKER: return launch_v<OP, SRC_WORKER>(src, p, rows, chunk, st);
    case SRC_SRV_IDENTITY: return launch_v<OP, SRC_SRV_IDENTITY>(src, p, rows, chunk, st);
    case SRC_SRV_SIGN1: return launch_v<OP, SRC_SRV_SIGN1>(src, p, rows, chunk, st);
    case SRC_SRV_TOPK: return launch_v<OP, SRC_SRV_TOPK>(src, p, rows, chunk, st);
    case SRC_SRV_QSGD: return launch_v<OP, SRC_SRV_QSGD>(src, p, rows, chunk, st);
    case SRC_SRV_CLIP: return launch_v<OP, SRC_SRV_CLIP>(src, p, rows, chunk, st);
    case SRC_SRV_RSPARSE: return launch_v<OP, SRC_SRV_RSPARSE>(src, p, rows, chunk, st);
    case SRC_WORKER_PLAIN: return launch_v<OP, SRC_WORKER_PLAIN>(src, p, rows, chunk, st);
    case SRC_SRV_TERNARY: return launch_v<OP, SRC_SRV_TERNARY>(src, p, rows, chunk, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

}  // namespace dsq
