// Operators whose scaling factor belongs to the WHOLE vector, fused with the error feedback:
//   - the 1-bit operator as Section 3.2 ("1-Bit Quantization") and Section 5.1 ("1-bit compression")
//     state it: sign(v) times magnitude(v) / magnitude(sign(v)), one factor per vector;
//   - the ternary quantiser of Section 5.1 ("Implementations and setups", item 2): with m the largest
//     magnitude of the vector an entry e survives as sign(e) with probability |e|/|m|, and one factor
//     magnitude(v) / magnitude(ternary vector) multiplies the result.
//
// The factor needs a sum over all d entries before the first residual can be written, so a pass is a
// chain of kernels.  Where an error is kept, the first kernel forms v (Eq. 2 on a worker, Eq. 4 on the
// server) and leaves it in the error buffer, which the last kernel overwrites with the residual; the
// kernels in between read v from there (source SRC_STORED: 4 bytes per entry instead of the 8 of a
// worker's g and delta, and no second or third decoding of the n payloads on the server).  Without
// an error buffer (no compensation) v is recomputed from its source in every kernel.
//
//   1-bit:    reduce (tile sums of |v| or v*v) -> finalize (factor) -> sign (words, residual, update)
//   ternary:  reduce (tile sums of |v|, tile maxima) -> finalize (||v||_1, m) -> draw (sign and
//             non-zero words, survivors per tile) -> finalize (factor) -> apply (residual, update)
//
// Summation order: pairwise in index order over the vector padded with zeros to the next power of
// two.  A tile is 4096 aligned entries, summed by the same tree as a 4096-entry chunk of the chunk
// kernels; the tile sums are then combined pairwise in tile order.  Counting survivors and taking
// maxima are exact in any order.
#include "dsq_chunked.cuh"

namespace dsq {

namespace {

constexpr uint64_t kWTile = 4096;   // entries per CTA: thread t holds float4 number j at entries (j*256 + t)*4

// Per-vector results of the finalize kernels.
struct WholeFin {
  float sum;     // ||v||_1 (or sum of squares for the 1-bit operator with l2 magnitudes)
  float vmax;    // ternary: largest magnitude
  float factor;  // the scaling factor that multiplies the sign / ternary vector
  float pad;
};

struct WholeScratch {
  float* part_sum;     // [rows, ntile]
  uint32_t* part_aux;  // [rows, ntile]: tile maxima as bit patterns, later survivors per tile
  WholeFin* fin;       // [rows]
  uint64_t ntile;
};

// The calling CTA's tile of vector `row`: v[j], and cnt[j] = how many of its four entries exist.
template <int SRC, bool FULL>
__device__ __forceinline__ void load_tile(const SrcParams& src, uint32_t row, uint64_t base, float4 (&v)[4], uint32_t (&cnt)[4]) {
  const uint32_t tid = threadIdx.x;
  const uint64_t d = src.d;
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
  } else if constexpr (FULL && SRC == SRC_STORED) {
    const float4* vp = reinterpret_cast<const float4*>(src.delta + (uint64_t)row * d + base) + tid;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      cnt[j] = 4;
      v[j] = vp[j * kThreads];
    }
  } else {
    uint64_t e[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      e[j] = base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = FULL ? 4u : (e[j] < d ? (uint32_t)min((uint64_t)4, d - e[j]) : 0u);
    }
    src_load_tile<SRC, 4>(src, row, e, cnt, v);
  }
}

// Sum over the CTA of one unsigned value per thread (all threads get it); MAX: the maximum instead.
template <bool MAX>
__device__ __forceinline__ uint32_t cta_reduce_u32(uint32_t x, uint32_t* s_w) {
  const uint32_t lane = threadIdx.x & 31u, wrp = threadIdx.x >> 5;
  x = MAX ? __reduce_max_sync(0xffffffffu, x) : __reduce_add_sync(0xffffffffu, x);
  __syncthreads();  // s_w may still be read from an earlier call
  if (lane == 0) s_w[wrp] = x;
  __syncthreads();
  uint32_t r = 0;
#pragma unroll
  for (uint32_t w = 0; w < kThreads / 32; ++w) r = MAX ? max(r, s_w[w]) : r + s_w[w];
  return r;
}

// ---------------------------------------------------------------- tile sums (and maxima)
// MODE 0: sum |v|;  1: sum v*v;  2: sum |v| and max |v|.
template <int SRC, int MODE, bool FULL>
__device__ __forceinline__ void reduce_body(const SrcParams& src, const WholeScratch& ws, float* v_store, float* s_red,
                                            uint32_t* s_w) {
  const uint32_t row = blockIdx.y;
  const uint64_t tile = blockIdx.x;
  float4 v[4];
  uint32_t cnt[4];
  load_tile<SRC, FULL>(src, row, tile * kWTile, v, cnt);
  if (v_store) {
    // v for the kernels that follow
    float* vr = v_store + (uint64_t)row * src.d;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = tile * kWTile + (uint64_t)(j * kThreads + threadIdx.x) * 4u;
      if (FULL || (src.vec && cnt[j] == 4)) {
        *reinterpret_cast<float4*>(vr + e) = v[j];
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)k < cnt[j]) vr[e + k] = compc(v[j], k);
      }
    }
  }
  float part[4];
  uint32_t mx = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float m0, m1, m2, m3;
    if constexpr (MODE == 1) {
      const float4 sq = mul4_rn(v[j], v[j]);
      m0 = sq.x; m1 = sq.y; m2 = sq.z; m3 = sq.w;
    } else {
      m0 = fabsf(v[j].x); m1 = fabsf(v[j].y); m2 = fabsf(v[j].z); m3 = fabsf(v[j].w);
      // the order of non-negative floats is the order of their bit patterns
      if (MODE == 2) mx = max(mx, max(max(__float_as_uint(m0), __float_as_uint(m1)), max(__float_as_uint(m2), __float_as_uint(m3))));
    }
    part[j] = __fadd_rn(__fadd_rn(m0, m1), __fadd_rn(m2, m3));
  }
  const float total = chunk_total<4, 8>(part, s_red);
  if constexpr (MODE == 2) mx = cta_reduce_u32<true>(mx, s_w);
  if (threadIdx.x == 0) {
    ws.part_sum[(uint64_t)row * ws.ntile + tile] = total;
    if (MODE == 2) ws.part_aux[(uint64_t)row * ws.ntile + tile] = mx;
  }
}

template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm) k_whole_reduce(const SrcParams src,
                                                                                                       const WholeScratch ws,
                                                                                                       float* v_store) {
  // v_store: NULL, or [rows, d] where v is left for the kernels that follow (it may be the buffer v's
  // error term was just read from: a thread writes only the entries it has read)
  pdl_prologue();
  __shared__ float s_red[64];
  __shared__ uint32_t s_w[kThreads / 32];
  if (src.vec && ((uint64_t)blockIdx.x + 1) * kWTile <= src.d) reduce_body<SRC, MODE, true>(src, ws, v_store, s_red, s_w);
  else reduce_body<SRC, MODE, false>(src, ws, v_store, s_red, s_w);
}

// ---------------------------------------------------------------- combining the tile results
// One 1024-thread CTA per vector.
//   PHASE 0 (1-bit): pairwise sum of the tile sums -> factor = sum / d, or sqrt(sum) / sqrt(d) with l2
//   PHASE 1 (ternary, after reduce): pairwise sum of the tile sums and the maximum of the tile maxima
//   PHASE 2 (ternary, after draw): survivors counted -> factor = ||v||_1 / survivors (0 if none)
template <int PHASE>
__global__ void __launch_bounds__(1024) k_whole_finalize(const WholeScratch ws, uint64_t d, uint32_t l2, float* out_scale,
                                                         uint64_t word_stride) {
  pdl_prologue();
  __shared__ float s_f[32];
  __shared__ uint32_t s_u[32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5, row = blockIdx.x;
  const uint64_t nt = ws.ntile;
  WholeFin* fin = ws.fin + row;
  if constexpr (PHASE == 2) {
    const uint32_t* pc = ws.part_aux + (uint64_t)row * nt;
    uint32_t c = 0;
    for (uint64_t i = tid; i < nt; i += 1024) c += pc[i];
    c = __reduce_add_sync(0xffffffffu, c);
    if (lane == 0) s_u[wrp] = c;
    __syncthreads();
    if (tid == 0) {
      uint32_t count = 0;
      for (int w = 0; w < 32; ++w) count += s_u[w];
      const float s = count ? __fdiv_rn(fin->sum, (float)count) : 0.f;
      fin->factor = s;
      out_scale[(uint64_t)row * word_stride] = s;
    }
    return;
  }
  // pairwise sum of ps[0..nt) padded with zeros to P = next power of two: thread t sums the aligned
  // block of B = P / 1024 consecutive tile sums (a binary counter of partial sums reproduces the
  // balanced tree), then the 1024 block sums are combined by butterflies in thread order
  const float* ps = ws.part_sum + (uint64_t)row * nt;
  uint64_t P = 1;
  while (P < nt) P <<= 1;
  float x = 0.f;
  if (P <= 1024) {
    if (tid < nt) x = ps[tid];
  } else {
    const uint64_t B = P >> 10, first = (uint64_t)tid * B;
    float stack[24];
#pragma unroll
    for (int l = 0; l < 24; ++l) stack[l] = 0.f;
    for (uint64_t i = 0; i < B; ++i) {
      float a = first + i < nt ? ps[first + i] : 0.f;
      int l = 0;
      for (; (i >> l) & 1u; ++l) a = __fadd_rn(stack[l], a);
      stack[l] = a;
    }
    int top = 0;
    while ((1ull << top) < B) ++top;
    x = stack[top];
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) x = __fadd_rn(x, __shfl_xor_sync(0xffffffffu, x, o));
  if (lane == 0) s_f[wrp] = x;
  uint32_t mx = 0;
  if constexpr (PHASE == 1) {
    const uint32_t* pm = ws.part_aux + (uint64_t)row * nt;
    for (uint64_t i = tid; i < nt; i += 1024) mx = max(mx, pm[i]);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) s_u[wrp] = mx;
  }
  __syncthreads();
  if (wrp != 0) return;
  float y = s_f[lane];
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) y = __fadd_rn(y, __shfl_xor_sync(0xffffffffu, y, o));
  if (PHASE == 1) mx = __reduce_max_sync(0xffffffffu, s_u[lane]);
  if (lane != 0) return;
  if (PHASE == 0) {
    // magnitude of v over magnitude of sign(v): ||v||_1 / d, or ||v||_2 / sqrt(d)
    const float s = l2 ? __fdiv_rn(__fsqrt_rn(y), __fsqrt_rn((float)d)) : __fdiv_rn(y, (float)d);
    fin->sum = y;
    fin->factor = s;
    out_scale[(uint64_t)row * word_stride] = s;
  } else {
    fin->sum = y;
    fin->vmax = __uint_as_float(mx);
  }
}

// ---------------------------------------------------------------- encoding with the factor known
// Stores the sign words (and, ternary, the non-zero words) of the calling CTA's tile.
__device__ __forceinline__ void store_tile_words(const uint32_t (&nib)[4], uint32_t* out_row, uint64_t base, uint64_t d) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t word = octet_sign_words<4>(nib, lane);
  const uint32_t r = lane & 7u;
  if (r < 4u) {
    const uint64_t e0 = base + (uint64_t)(r * kThreads + (tid & ~7u)) * 4u;  // first entry of that word
    if (e0 < d) out_row[e0 >> 5] = word;
  }
}

// Residual v - C (unless no error is kept) and, on a fused server pass, x = x - gamma * C.
template <int SRC, bool FULL>
__device__ __forceinline__ void finish_entries(const SrcParams& src, const WholeParams& p, uint32_t row, uint64_t e, uint32_t cnt,
                                               float4 v, float4 C) {
  if (!cnt) return;
  if (SRC != SRC_WORKER_PLAIN && (SRC == SRC_WORKER || p.delta_out)) {
    const float4 dl = sub4_rn(v, C);
    float* drow = p.delta_out + (uint64_t)row * p.delta_row_stride;
    if constexpr (FULL) st_stream4(drow + e, dl);
    else store_row4(drow, e, cnt, src.vec, dl);
  }
  if (!is_worker_src(SRC) && p.x) {
    const float4 xo = load_row4(p.x, e, cnt, 1);
    float4 xn;  // scalar: a multiply that feeds a subtract must not be contracted
    xn.x = __fsub_rn(xo.x, __fmul_rn(p.gamma, C.x)); xn.y = __fsub_rn(xo.y, __fmul_rn(p.gamma, C.y));
    xn.z = __fsub_rn(xo.z, __fmul_rn(p.gamma, C.z)); xn.w = __fsub_rn(xo.w, __fmul_rn(p.gamma, C.w));
    store_row4(p.x, e, cnt, 1, xn);
  }
}

template <int SRC, bool FULL>
__device__ __forceinline__ void sign_body(const SrcParams& src, const WholeParams& p, const WholeScratch& ws) {
  const uint32_t row = blockIdx.y, tid = threadIdx.x;
  const uint64_t base = (uint64_t)blockIdx.x * kWTile;
  const float s = ws.fin[row].factor;
  float4 v[4];
  uint32_t cnt[4], nib[4];
  load_tile<SRC, FULL>(src, row, base, v, cnt);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float4 C;
    nib[j] = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool nonneg = compc(v[j], k) >= 0.f;
      nib[j] |= (nonneg ? 1u : 0u) << k;
      comp(C, k) = nonneg ? s : -s;
    }
    if constexpr (!FULL) nib[j] &= (1u << cnt[j]) - 1u;  // pad bits are 0
    finish_entries<SRC, FULL>(src, p, row, base + (uint64_t)(j * kThreads + tid) * 4u, cnt[j], v[j], C);
  }
  store_tile_words(nib, p.out_sgn + (uint64_t)row * p.word_stride, base, src.d);
}

template <int SRC>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm) k_whole_sign(const SrcParams src,
                                                                                                     const WholeParams p,
                                                                                                     const WholeScratch ws) {
  pdl_prologue();
  if (src.vec && ((uint64_t)blockIdx.x + 1) * kWTile <= src.d) sign_body<SRC, true>(src, p, ws);
  else sign_body<SRC, false>(src, p, ws);
}

// Ternary, first half: who survives.  Entry j draws u from word j % 4 of the Philox block with counter
// (j / 4, 0xFFFFFFFE, worker or 0xFFFFFFFF on the server pass, step) and survives iff u < |v_j| / m.
template <int SRC, bool FULL>
__device__ __forceinline__ void draw_body(const SrcParams& src, const WholeParams& p, const WholeScratch& ws, uint32_t* s_w) {
  const uint32_t row = blockIdx.y, tid = threadIdx.x;
  const uint64_t base = (uint64_t)blockIdx.x * kWTile;
  const float m = ws.fin[row].vmax;
  float4 v[4];
  uint32_t cnt[4], sgn[4], nz[4];
  load_tile<SRC, FULL>(src, row, base, v, cnt);
  uint32_t kept = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
    const uint4 rnd = philox4x32_10(make_uint4((uint32_t)(e >> 2), 0xFFFFFFFEu, p.server_pass ? 0xFFFFFFFFu : row, p.step), p.keys);
    const uint32_t w[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
    sgn[j] = 0;
    nz[j] = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float val = compc(v[j], k);
      const float u = __fmul_rn(__uint2float_rn(w[k] >> 8), 5.9604644775390625e-08f);  // 2^-24, exact
      const bool live = (FULL || (uint32_t)k < cnt[j]) && m > 0.f && u < __fdiv_rn(fabsf(val), m);
      sgn[j] |= (val >= 0.f ? 1u : 0u) << k;
      nz[j] |= (live ? 1u : 0u) << k;
    }
    if constexpr (!FULL) sgn[j] &= (1u << cnt[j]) - 1u;  // pad bits are 0
    kept += __popc(nz[j]);
  }
  store_tile_words(sgn, p.out_sgn + (uint64_t)row * p.word_stride, base, src.d);
  store_tile_words(nz, p.out_nz + (uint64_t)row * p.word_stride, base, src.d);
  kept = cta_reduce_u32<false>(kept, s_w);
  if (tid == 0) ws.part_aux[(uint64_t)row * ws.ntile + blockIdx.x] = kept;
}

template <int SRC>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm) k_whole_ternary_draw(const SrcParams src,
                                                                                                             const WholeParams p,
                                                                                                             const WholeScratch ws) {
  pdl_prologue();
  __shared__ uint32_t s_w[kThreads / 32];
  if (src.vec && ((uint64_t)blockIdx.x + 1) * kWTile <= src.d) draw_body<SRC, true>(src, p, ws, s_w);
  else draw_body<SRC, false>(src, p, ws, s_w);
}

// Ternary, second half: Q[v]_j = +-factor where the entry survived (its bit in the non-zero words this
// pass wrote), +0 elsewhere; residual and update.
template <int SRC, bool FULL>
__device__ __forceinline__ void apply_body(const SrcParams& src, const WholeParams& p, const WholeScratch& ws) {
  const uint32_t row = blockIdx.y, tid = threadIdx.x;
  const uint64_t base = (uint64_t)blockIdx.x * kWTile;
  const float s = ws.fin[row].factor;
  const uint32_t* nzrow = p.out_nz + (uint64_t)row * p.word_stride;
  float4 v[4];
  uint32_t cnt[4];
  load_tile<SRC, FULL>(src, row, base, v, cnt);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
    if (!FULL && !cnt[j]) continue;
    const uint32_t z = nzrow[e >> 5] >> (uint32_t)(e & 31u);
    float4 C;
#pragma unroll
    for (int k = 0; k < 4; ++k) comp(C, k) = ((z >> k) & 1u) ? (compc(v[j], k) >= 0.f ? s : -s) : 0.f;
    finish_entries<SRC, FULL>(src, p, row, e, cnt[j], v[j], C);
  }
}

template <int SRC>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) ? 0 : kServerCtasPerSm) k_whole_ternary_apply(const SrcParams src,
                                                                                                              const WholeParams p,
                                                                                                              const WholeScratch ws) {
  pdl_prologue();
  if (src.vec && ((uint64_t)blockIdx.x + 1) * kWTile <= src.d) apply_body<SRC, true>(src, p, ws);
  else apply_body<SRC, false>(src, p, ws);
}

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

}  // namespace

uint64_t whole_workspace_bytes(uint64_t d, uint32_t rows) {
  const uint64_t ntile = (d + kWTile - 1) / kWTile;
  return 2 * round16((uint64_t)rows * ntile * 4) + round16((uint64_t)rows * sizeof(WholeFin));
}

cudaError_t launch_whole(int op, int srck, const SrcParams& src, const WholeParams& p, void* workspace, uint32_t rows,
                         cudaStream_t st) {
  WholeScratch ws;
  ws.ntile = (src.d + kWTile - 1) / kWTile;
  uint8_t* w = static_cast<uint8_t*>(workspace);
  const uint64_t part_bytes = round16((uint64_t)rows * ws.ntile * 4);
  ws.part_sum = reinterpret_cast<float*>(w);
  ws.part_aux = reinterpret_cast<uint32_t*>(w + part_bytes);
  ws.fin = reinterpret_cast<WholeFin*>(w + 2 * part_bytes);
  const dim3 grid((unsigned)ws.ntile, rows, 1);
  // v can be left in the error buffer if the pass has one, reads its error term from it and writes rows d apart
  const bool stored = srck != SRC_WORKER_PLAIN && p.delta_out != nullptr && src.delta == p.delta_out &&
                      (rows == 1 || p.delta_row_stride == src.d);
  float* v_store = stored ? p.delta_out : nullptr;
  // the source of the kernels after the first
  const int srck2 = stored ? (int)SRC_STORED : srck;
#define DSQ_SWITCH_SRC2(X)                                   \
  if (srck2 == SRC_STORED) { X(SRC_STORED); } else { DSQ_SWITCH_SRC(srck2, X) }
  if (op == DS_Q_SIGN1) {
    if (p.l2) {
#define DSQ_W(S) launch_pdl(k_whole_reduce<S, 1>, grid, kThreads, st, src, ws, v_store)
      DSQ_SWITCH_SRC(srck, DSQ_W)
#undef DSQ_W
    } else {
#define DSQ_W(S) launch_pdl(k_whole_reduce<S, 0>, grid, kThreads, st, src, ws, v_store)
      DSQ_SWITCH_SRC(srck, DSQ_W)
#undef DSQ_W
    }
    launch_pdl(k_whole_finalize<0>, rows, 1024, st, ws, src.d, p.l2, p.out_scale, p.word_stride);
#define DSQ_W(S) launch_pdl(k_whole_sign<S>, grid, kThreads, st, src, p, ws)
    DSQ_SWITCH_SRC2(DSQ_W)
#undef DSQ_W
    count_launches(3);
    return cudaGetLastError();
  }
  if (op == DS_Q_TERNARY) {
#define DSQ_W(S) launch_pdl(k_whole_reduce<S, 2>, grid, kThreads, st, src, ws, v_store)
    DSQ_SWITCH_SRC(srck, DSQ_W)
#undef DSQ_W
    launch_pdl(k_whole_finalize<1>, rows, 1024, st, ws, src.d, 0u, p.out_scale, p.word_stride);
#define DSQ_W(S) launch_pdl(k_whole_ternary_draw<S>, grid, kThreads, st, src, p, ws)
    DSQ_SWITCH_SRC2(DSQ_W)
#undef DSQ_W
    launch_pdl(k_whole_finalize<2>, rows, 1024, st, ws, src.d, 0u, p.out_scale, p.word_stride);
#define DSQ_W(S) launch_pdl(k_whole_ternary_apply<S>, grid, kThreads, st, src, p, ws)
    DSQ_SWITCH_SRC2(DSQ_W)
#undef DSQ_W
    count_launches(5);
    return cudaGetLastError();
  }
#undef DSQ_SWITCH_SRC2
  return cudaErrorInvalidValue;
}

}  // namespace dsq
