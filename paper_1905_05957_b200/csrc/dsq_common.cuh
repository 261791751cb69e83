// Shared device-side pieces of the DoubleSqueeze kernels: parameter blocks, the "source" of the
// vector that is about to be compressed (worker: g + delta, Eq. 2; server: decoded mean of the
// worker payloads + delta, Eq. 4), and the Philox4x32-10 generator.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsq {

constexpr int kThreads = 256;  // every streaming kernel uses 256-thread CTAs

// Kernels that decode worker payloads (server passes) are compiled for this many CTAs per SM: they
// are bound by instruction issue and by the latency of the payload loads, and four resident CTAs
// serve both better than a larger register budget does (measured on all server kernels).
constexpr int kServerCtasPerSm = 4;

// Kernels are launched with programmatic stream serialization: once every CTA of a kernel has
// passed launch_dependents (or left), the CTAs of the next kernel in the stream may take free
// slots; there they stop at wait until the earlier kernel has completed and its writes are
// visible.  Every kernel starts with this prologue, so nothing before it touches memory.
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

enum Src : int {
  SRC_WORKER = 0,        // v = g[row] + delta_w[row]
  SRC_SRV_IDENTITY = 1,  // v = (sum_i c_i) * inv_n + delta_s
  SRC_SRV_SIGN1 = 2,
  SRC_SRV_TOPK = 3,      // the sparse payloads were summed into a dense accumulator beforehand
  SRC_SRV_QSGD = 4,
  SRC_SRV_CLIP = 5,      // payload = the high bits of every entry
  SRC_SRV_RSPARSE = 6,   // payload = the survivors of every chunk and the chunk's draw
  SRC_WORKER_PLAIN = 7,  // v = g[row]: a worker that keeps no error (no compensation)
  SRC_SRV_TERNARY = 8,   // payload = sign words, non-zero words and one factor per worker
  SRC_STORED = 9,        // v = delta[row]: an earlier kernel of the same pass formed v and left it where the error lives
                         // (operators with one factor per vector only; not part of DSQ_SWITCH_SRC)
};

__host__ __device__ constexpr bool is_worker_src(int src) { return src == SRC_WORKER || src == SRC_WORKER_PLAIN; }

// Where v comes from.  Worker payload sub-arrays follow the documented payload layout.
struct SrcParams {
  const float* g;          // worker: gradients [n, d]
  const float* delta;      // worker: delta_w [n, d]; server: delta_s [d], or NULL: no error is carried (v is the plain mean)
  uint64_t d;
  uint32_t n;              // server: number of payloads to average
  float inv_n;             // server: 1/n rounded once
  const uint8_t* wp;       // server: base of the n worker payloads
  uint64_t wp_stride;      // bytes between payloads
  uint64_t wp_off[3];      // sub-array offsets inside a payload
  uint32_t w_log2_chunk;   // worker chunk length (SIGN1, QSGD)
  float w_levels;          // worker QSGD level count as a float
  uint32_t w_clip_bits;    // worker CLIP: low bits that were set to zero (16 or 24)
  uint32_t w_log2_keep;    // worker RSPARSE: log2 S (one entry in S survives)
  const float* acc;        // SRC_SRV_TOPK: dense accumulator [d] holding the sum of the sparse payloads
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
  } else if (cnt) {
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

// Packed pairs of binary32 (sm_100 adds .f32x2 arithmetic: one instruction, two IEEE results, each
// rounded on its own exactly like the scalar instruction).  A pair lives in a 64-bit register.
// Never let a packed multiply feed a packed add or subtract directly: that pair was observed to be
// contracted into a fused multiply-add, which changes the rounding; such spots stay scalar.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 r, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r)); }
__device__ __forceinline__ f32x2 add2_rn(f32x2 a, f32x2 b) { f32x2 d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 add2_rz(f32x2 a, f32x2 b) { f32x2 d; asm("add.rz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 sub2_rn(f32x2 a, f32x2 b) { f32x2 d; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 mul2_rn(f32x2 a, f32x2 b) { f32x2 d; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ float4 add4_rn(float4 a, float4 b) {
  float4 r;
  unpack2(add2_rn(pack2(a.x, a.y), pack2(b.x, b.y)), r.x, r.y);
  unpack2(add2_rn(pack2(a.z, a.w), pack2(b.z, b.w)), r.z, r.w);
  return r;
}
__device__ __forceinline__ float4 sub4_rn(float4 a, float4 b) {
  float4 r;
  unpack2(sub2_rn(pack2(a.x, a.y), pack2(b.x, b.y)), r.x, r.y);
  unpack2(sub2_rn(pack2(a.z, a.w), pack2(b.z, b.w)), r.z, r.w);
  return r;
}
__device__ __forceinline__ float4 mul4_rn(float4 a, float4 b) {
  float4 r;
  unpack2(mul2_rn(pack2(a.x, a.y), pack2(b.x, b.y)), r.x, r.y);
  unpack2(mul2_rn(pack2(a.z, a.w), pack2(b.z, b.w)), r.z, r.w);
  return r;
}

// +m or -m according to bit `k` of the sign word `w` (1 = non-negative), without a branch.
__device__ __forceinline__ float signed_by_bit(float m, uint32_t w, int k) {
  return __uint_as_float(__float_as_uint(m) ^ ((~w << (31 - k)) & 0x80000000u));
}

// Exact float value of byte `k` of `x` (one conversion instruction with a byte selector).
__device__ __forceinline__ float byte_to_float(uint32_t x, int k) { return __uint2float_rn((x >> (8 * k)) & 0xFFu); }

// The vector to compress, for a tile of V rows: row j of the calling thread is the float4 at entry
// e[j] of vector `row`; cnt[j] in [0, 4] says how many of its entries exist (the others, and whole
// rows with cnt 0, are returned as +0).  Must be called by all 32 lanes of a warp together, the
// lanes holding consecutive float4 of each row (e[j] = 128-aligned warp base + 4 * lane): server
// sources load the sign words and scales of eight workers with one instruction per row (lane l
// fetches word l%4 of worker l/4) and hand them round with shuffles.  Workers are accumulated in
// order 0..n-1, the order in which Eq. 4 is summed.
template <int SRC, int V>
__device__ __forceinline__ void src_load_tile(const SrcParams& p, uint32_t row, const uint64_t (&e)[V],
                                              const uint32_t (&cnt)[V], float4 (&v)[V]) {
  if constexpr (SRC == SRC_WORKER) {
    const uint64_t off = (uint64_t)row * p.d;
    float4 a[V], b[V];
#pragma unroll
    for (int j = 0; j < V; ++j) a[j] = load_row4(p.g + off, e[j], cnt[j], p.vec);
#pragma unroll
    for (int j = 0; j < V; ++j) b[j] = load_row4(p.delta + off, e[j], cnt[j], p.vec);
#pragma unroll
    for (int j = 0; j < V; ++j)
      v[j] = add4_rn(a[j], b[j]);
  } else if constexpr (SRC == SRC_WORKER_PLAIN) {
    const uint64_t off = (uint64_t)row * p.d;
#pragma unroll
    for (int j = 0; j < V; ++j) v[j] = load_row4(p.g + off, e[j], cnt[j], p.vec);
  } else if constexpr (SRC == SRC_STORED) {
    // written by the previous kernel of the chain: ordinary loads
    const float* vr = p.delta + (uint64_t)row * p.d;
#pragma unroll
    for (int j = 0; j < V; ++j) {
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (p.vec && cnt[j] == 4) {
        v[j] = *reinterpret_cast<const float4*>(vr + e[j]);
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k < cnt[j]) comp(v[j], k) = vr[e[j] + k];
      }
    }
  } else {
    const uint32_t lane = threadIdx.x & 31u;
    float4 acc[V], ds[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
      acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      ds[j] = p.delta ? load_row4(p.delta, e[j], cnt[j], p.vec) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if constexpr (SRC == SRC_SRV_IDENTITY) {
      for (uint32_t i = 0; i < p.n; ++i) {
        const float* c = reinterpret_cast<const float*>(p.wp + i * p.wp_stride + p.wp_off[0]);
        float4 ci[V];
#pragma unroll
        for (int j = 0; j < V; ++j) ci[j] = load_row4(c, e[j], cnt[j], 1);
#pragma unroll
        for (int j = 0; j < V; ++j) {
          acc[j] = add4_rn(acc[j], ci[j]);
        }
      }
    } else if constexpr (SRC == SRC_SRV_SIGN1 || SRC == SRC_SRV_QSGD || SRC == SRC_SRV_TERNARY) {
      constexpr int kSgn = SRC == SRC_SRV_QSGD ? 1 : 0;     // payload sub-array of the sign words
      constexpr int kScl = SRC == SRC_SRV_SIGN1 ? 1 : 2;    // ... of the per-chunk scale / grid step / factor
      const uint64_t nw = (p.d + 31) >> 5;
      const uint32_t sh = (lane & 7u) * 4u;                 // this lane's nibble inside its word
      for (uint32_t i0 = 0; i0 < p.n; i0 += 8) {
        uint32_t wreg[V];
        uint32_t zreg[SRC == SRC_SRV_TERNARY ? V : 1];      // ternary: words of the non-zero plane
        float sreg[V];
        uint32_t lv[SRC == SRC_SRV_QSGD ? V : 1][SRC == SRC_SRV_QSGD ? 8 : 1];
#pragma unroll
        for (int j = 0; j < V; ++j) {
          // warp base of this row: entry of lane 0 (valid arithmetic even where the row is past the end)
          const uint64_t e0 = e[j] - 4u * lane;
          const uint64_t word = (e0 >> 5) + (lane & 3u);
          const uint32_t wi = i0 + (lane >> 2);
          wreg[j] = 0;
          sreg[j] = 0.f;
          if (wi < p.n && word < nw)
            wreg[j] = __ldg(reinterpret_cast<const uint32_t*>(p.wp + wi * p.wp_stride + p.wp_off[kSgn]) + word);
          if constexpr (SRC == SRC_SRV_TERNARY) {
            zreg[j] = 0;
            if (wi < p.n && word < nw)
              zreg[j] = __ldg(reinterpret_cast<const uint32_t*>(p.wp + wi * p.wp_stride + p.wp_off[1]) + word);
          }
          if (lane < 8 && i0 + lane < p.n && e0 < p.d)
            sreg[j] = __ldg(reinterpret_cast<const float*>(p.wp + (i0 + lane) * p.wp_stride + p.wp_off[kScl]) +
                            (e0 >> p.w_log2_chunk));
          if constexpr (SRC == SRC_SRV_QSGD) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              lv[j][u] = 0;
              if (i0 + u < p.n && cnt[j])
                lv[j][u] = __ldcs(reinterpret_cast<const uint32_t*>(p.wp + (i0 + u) * p.wp_stride + p.wp_off[0] + e[j]));
            }
          }
        }
#pragma unroll
        for (int j = 0; j < V; ++j) {
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t ww = __shfl_sync(0xffffffffu, wreg[j], u * 4 + (lane >> 3)) >> sh;
            const float sc = __shfl_sync(0xffffffffu, sreg[j], u);
            if (i0 + u < p.n) {
              if constexpr (SRC == SRC_SRV_SIGN1) {
                acc[j] = add4_rn(acc[j], make_float4(signed_by_bit(sc, ww, 0), signed_by_bit(sc, ww, 1),
                                                     signed_by_bit(sc, ww, 2), signed_by_bit(sc, ww, 3)));
              } else if constexpr (SRC == SRC_SRV_TERNARY) {
                // +-factor where the entry's non-zero bit is set, +0 elsewhere
                const uint32_t zz = __shfl_sync(0xffffffffu, zreg[j], u * 4 + (lane >> 3)) >> sh;
                acc[j] = add4_rn(acc[j], make_float4((zz & 1u) ? signed_by_bit(sc, ww, 0) : 0.f, (zz & 2u) ? signed_by_bit(sc, ww, 1) : 0.f,
                                                     (zz & 4u) ? signed_by_bit(sc, ww, 2) : 0.f, (zz & 8u) ? signed_by_bit(sc, ww, 3) : 0.f));
              } else {
                const uint32_t l4 = lv[j][u];
                const float4 mag = mul4_rn(make_float4(byte_to_float(l4, 0), byte_to_float(l4, 1), byte_to_float(l4, 2),
                                                       byte_to_float(l4, 3)),
                                           make_float4(sc, sc, sc, sc));
                acc[j] = add4_rn(acc[j], make_float4(signed_by_bit(mag.x, ww, 0), signed_by_bit(mag.y, ww, 1),
                                                     signed_by_bit(mag.z, ww, 2), signed_by_bit(mag.w, ww, 3)));
              }
            }
          }
        }
      }
    } else if constexpr (SRC == SRC_SRV_CLIP) {
      // Q[v_i] = hi << bits; four workers' rows are fetched before they are added (in worker order)
      const bool wide = p.w_clip_bits == 16;  // 16-bit entries, else 8-bit
      for (uint32_t i0 = 0; i0 < p.n; i0 += 4) {
        uint2 raw[V][4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint8_t* hp = p.wp + (uint64_t)(i0 + u) * p.wp_stride + p.wp_off[0];
#pragma unroll
          for (int j = 0; j < V; ++j) {
            raw[j][u] = make_uint2(0u, 0u);
            if (i0 + u >= p.n || !cnt[j]) continue;
            if (cnt[j] == 4) {
              if (wide) raw[j][u] = __ldcs(reinterpret_cast<const uint2*>(hp + 2 * e[j]));
              else raw[j][u].x = __ldcs(reinterpret_cast<const uint32_t*>(hp + e[j]));
            } else {
              // a ragged last row: entry by entry, packed as a full row would be
              uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
              for (int k = 0; k < 4; ++k)
                if ((uint32_t)k < cnt[j])
                  w[k] = wide ? (uint32_t)__ldcs(reinterpret_cast<const uint16_t*>(hp + 2 * e[j]) + k) : (uint32_t)__ldcs(hp + e[j] + k);
              raw[j][u] = wide ? make_uint2(w[0] | w[1] << 16, w[2] | w[3] << 16)
                               : make_uint2(w[0] | w[1] << 8 | w[2] << 16 | w[3] << 24, 0u);
            }
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (i0 + u < p.n) {
#pragma unroll
            for (int j = 0; j < V; ++j) {
              const uint2 r = raw[j][u];
              float4 c;
              if (wide) {
                c = make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u),
                                __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xFFFF0000u));
              } else {
                c = make_float4(__uint_as_float(r.x << 24), __uint_as_float((r.x << 16) & 0xFF000000u),
                                __uint_as_float((r.x << 8) & 0xFF000000u), __uint_as_float(r.x & 0xFF000000u));
              }
              acc[j] = add4_rn(acc[j], c);
            }
          }
        }
      }
    } else if constexpr (SRC == SRC_SRV_RSPARSE) {
      // entry j of worker i survives iff (offset of j in its chunk) mod S equals the chunk's draw o_i;
      // its value sits in slot j / S.  With S >= 4 the four entries of a float4 lie in one group of S,
      // so a worker has at most ONE survivor among them: it is there iff o_i agrees with the entries'
      // offset in everything but the low two bits, it is component o_i % 4, and its slot is the
      // group's.  Eight workers at a time: their draws are fetched together, then their survivors,
      // then they are added in worker order.
      const uint32_t smask = (1u << p.w_log2_keep) - 1u;
      if (p.w_log2_keep >= 2) {
        for (uint32_t i0 = 0; i0 < p.n; i0 += 8) {
          uint32_t o[V][8];
          float c[V][8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t* off = reinterpret_cast<const uint32_t*>(p.wp + (uint64_t)(i0 + u) * p.wp_stride + p.wp_off[1]);
#pragma unroll
            for (int j = 0; j < V; ++j) o[j][u] = (i0 + u < p.n && cnt[j]) ? __ldg(off + (e[j] >> p.w_log2_chunk)) : 0xFFFFFFFFu;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float* val = reinterpret_cast<const float*>(p.wp + (uint64_t)(i0 + u) * p.wp_stride + p.wp_off[0]);
#pragma unroll
            for (int j = 0; j < V; ++j) {
              // the filler 0xFFFFFFFF is no draw (draws are at most S - 1); a survivor past the end of a ragged
              // last float4 reads its slot, which holds +0, and is dropped by the masking of v below anyway
              const bool mine = o[j][u] <= smask && ((((uint32_t)e[j] ^ o[j][u]) & smask & ~3u) == 0u);
              c[j][u] = mine ? __ldg(val + (e[j] >> p.w_log2_keep)) : 0.f;
            }
          }
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (i0 + u < p.n) {
#pragma unroll
              for (int j = 0; j < V; ++j) {
                const uint32_t k = o[j][u] & 3u;
                // adding +0 to the other three components changes nothing: acc is never -0
                acc[j] = add4_rn(acc[j], make_float4(k == 0u ? c[j][u] : 0.f, k == 1u ? c[j][u] : 0.f, k == 2u ? c[j][u] : 0.f,
                                                     k == 3u ? c[j][u] : 0.f));
              }
            }
        }
      } else {
        // S = 2: two survivors per float4; four workers at a time, entry by entry
        for (uint32_t i0 = 0; i0 < p.n; i0 += 4) {
          uint32_t o[V][4];
          float4 c[V][4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t* off = reinterpret_cast<const uint32_t*>(p.wp + (uint64_t)(i0 + u) * p.wp_stride + p.wp_off[1]);
#pragma unroll
            for (int j = 0; j < V; ++j) o[j][u] = (i0 + u < p.n && cnt[j]) ? __ldg(off + (e[j] >> p.w_log2_chunk)) : 0xFFFFFFFFu;
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float* val = reinterpret_cast<const float*>(p.wp + (uint64_t)(i0 + u) * p.wp_stride + p.wp_off[0]);
#pragma unroll
            for (int j = 0; j < V; ++j) {
              c[j][u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int k = 0; k < 4; ++k)
                if ((uint32_t)k < cnt[j] && (((uint32_t)e[j] + k) & smask) == o[j][u])   // never true for the filler 0xFFFFFFFF
                  comp(c[j][u], k) = __ldg(val + ((e[j] + k) >> p.w_log2_keep));
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (i0 + u < p.n) {
#pragma unroll
              for (int j = 0; j < V; ++j) acc[j] = add4_rn(acc[j], c[j][u]);
            }
        }
      }
    } else {  // SRC_SRV_TOPK: the sparse payloads were summed into p.acc (cleared before every use)
#pragma unroll
      for (int j = 0; j < V; ++j) acc[j] = load_row4(p.acc, e[j], cnt[j], p.vec);
    }
#pragma unroll
    for (int j = 0; j < V; ++j) {
      // scalar on purpose: a packed multiply feeding a packed add was seen to come out fused
      if (p.delta) {
        v[j].x = __fadd_rn(__fmul_rn(acc[j].x, p.inv_n), ds[j].x); v[j].y = __fadd_rn(__fmul_rn(acc[j].y, p.inv_n), ds[j].y);
        v[j].z = __fadd_rn(__fmul_rn(acc[j].z, p.inv_n), ds[j].z); v[j].w = __fadd_rn(__fmul_rn(acc[j].w, p.inv_n), ds[j].w);
      } else {  // no error is carried: the plain mean, with no addition at all
        v[j].x = __fmul_rn(acc[j].x, p.inv_n); v[j].y = __fmul_rn(acc[j].y, p.inv_n);
        v[j].z = __fmul_rn(acc[j].z, p.inv_n); v[j].w = __fmul_rn(acc[j].w, p.inv_n);
      }
      // entries past the end must read as +0 whatever the payload padding holds
      if (cnt[j] < 4) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k >= cnt[j]) comp(v[j], k) = 0.f;
      }
    }
  }
}

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors.  The key
// of round r is key + r * (0x9E3779B9, 0xBB67AE85); the twenty round-key words are computed once
// on the host (philox_key_schedule) and read from the kernel parameters.
struct PhiloxKeys {
  uint32_t k[10][2];
};

__host__ __device__ inline PhiloxKeys philox_key_schedule(uint32_t k0, uint32_t k1) {
  PhiloxKeys ks;
  for (int r = 0; r < 10; ++r) {
    ks.k[r][0] = k0 + (uint32_t)r * 0x9E3779B9u;
    ks.k[r][1] = k1 + (uint32_t)r * 0xBB67AE85u;
  }
  return ks;
}

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const PhiloxKeys& ks) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c.x;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c.z;
    c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ ks.k[r][0], (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ ks.k[r][1],
                   (uint32_t)p0);
  }
  return c;
}

}  // namespace dsq
