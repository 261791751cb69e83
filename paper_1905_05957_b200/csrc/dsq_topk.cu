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
//              while v is still in registers, writes (value bits, index) of every entry with
//              key >= lo into the tile's own region of the list, in index order (one region of
//              4096 slots per 4096-entry tile, so CTAs never reserve space from each other).
//              Entries above the band (key > hi) are kept whatever tau turns out to be: they are
//              counted and already zeroed in the residual.  tile_info = (listed, above, 0, 0).
//   lhist 1    copies the entries inside the band (the candidates) out of the regions into one
//              dense (key, index) list and counts the top 12 key bits on the way; accepts the
//              prediction only if the k-th entry is a candidate (above < k <= above + candidates)
//   hist       only after a miss (or without history): entries zeroed by pass1 are restored from
//              the regions, then a full 4096-bin histogram of v is counted
//   mark       only after a miss: the exact bin tb from that histogram; re-read v, rebuild the
//              regions and the dense list for that bin
//   lhist 2,3  the next 12, then the last 7 key bits from the dense list: tau and r
//   classify   every candidate with key >= tau adds one to its tile's counters in tile_info
//              (.z: above tau, .w: equal to tau)
//              and the last CTA of a vector takes the exclusive prefix over the tiles of (above the
//              band + above tau, ties) and checks that exactly k entries will be emitted
//   emit       a warp per tile walks the region in index order; the prefix gives the tile's first
//              output slot, ballots place the kept entries: write (index, value), zero the kept
//              candidates in delta (delta = v - Q[v], Eq. 3), and on a fused server pass update x
// In the steady state v is read once and written once; the kernels marked "only after a miss"
// leave at once.  A wrong, missing or garbage history costs time, never correctness.
//
// Pipeline without a list (built-in-scratch entry point, whose scratch must stay small):
//   pass1 (full histogram) -> pick -> mark (kept + candidate bitmaps) -> refine, pick, refine, pick
//   (candidates gathered through their bitmap) -> finalize -> scan -> emit.
//
// No float atomics, no spinning; integer atomics commute and output slots come from prefix sums
// over index-ordered regions or bitmaps, so the result does not depend on scheduling.
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
constexpr uint32_t kBandHalf = 1u << 13;           // least half-width of the band in key units (0.07 % of magnitude)
constexpr uint32_t kMaxErr = 1u << 21;             // widest extrapolation error followed (band: half an octave each way)
constexpr uint32_t kFirstErr = kMaxErr;            // error assumed before any extrapolation has been checked
constexpr int kMaxTrend = 1 << 20;                 // largest step-to-step drift that is extrapolated (9 %)

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }

// Keys are monotone in log-magnitude (2^23 units per octave), so a threshold that drifts by a
// steady factor moves by a steady key difference.  The band is the last threshold, extrapolated by
// the last change (the drift itself changes slowly), widened on both sides by the largest of a
// quarter of that change, 0.07 % of magnitude, and twice the recent extrapolation error (a decaying
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

// ================================================================ list pipeline

// ---------------------------------------------------------------- marking a tile
// One 4096-entry tile held by a 256-thread CTA: thread t has the float4 groups at entries
// base + (j * 256 + t) * 4, j < 4 (cnt[j] of each inside the vector).  Every entry with key >= lo
// is "listed": its (value bits, index) goes to the tile's own region of the list (kTile slots,
// enough for the whole tile, so CTAs never share a region), in index order.  Listed entries with
// key > hi are certain to be kept; they are counted and already zeroed in the residual (their
// value survives in the list).  info receives (listed, above hi, 0, 0); the two zeros are the
// counters classify fills.  out_row = NULL: nothing is zeroed.  s_tot: one uint4 per warp, free for reuse after the call's barrier
// has been passed by all threads a second time.  Called by all threads of the CTA.
template <bool FULL>
__device__ __forceinline__ void mark_tile(const float4 (&v)[4], const uint32_t (&cnt)[4], uint64_t base, uint32_t key_lo,
                                          uint32_t key_hi, float* out_row, uint2* region, uint4* info, uint4* s_tot) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5;
  uint32_t sel[4], kept = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    sel[j] = 0;
    const uint32_t k0 = key_of(v[j].x), k1 = key_of(v[j].y), k2 = key_of(v[j].z), k3 = key_of(v[j].w);
    if (max(max(k0, k1), max(k2, k3)) >= key_lo) {
      // only groups with a listed entry get in here
      uint32_t gt = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t key = key_of(compc(v[j], k));
        if (FULL || (uint32_t)k < cnt[j]) {  // entries past the end were loaded as +0 and are no entries
          if (key >= key_lo) sel[j] |= 1u << k;
          if (key > key_hi) gt |= 1u << k;
        }
      }
      if (gt) {
        if (out_row) {  // NULL: no error is kept (v is the caller's gradient, which is never written)
          float* o = out_row + base + (uint64_t)(j * kThreads + tid) * 4u;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if ((gt >> k) & 1u) o[k] = 0.f;  // delta = v - Q[v] at an entry that is kept whatever tau turns out to be
        }
        kept += __popc(gt);
      }
    }
  }
  // index order is (j, thread, k): per-j counts, packed two to a word, scanned over the warp
  const uint32_t ca = __popc(sel[0]) | (__popc(sel[1]) << 16), cb = __popc(sel[2]) | (__popc(sel[3]) << 16);
  uint32_t ia = ca, ib = cb;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t ya = __shfl_up_sync(0xffffffffu, ia, o), yb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= (uint32_t)o) { ia += ya; ib += yb; }
  }
  kept = __reduce_add_sync(0xffffffffu, kept);
  if (lane == 31) s_tot[wrp] = make_uint4(ia, ib, kept, 0u);
  __syncthreads();
  uint32_t sa = 0, sb = 0, pa = 0, pb = 0, kt = 0;
#pragma unroll
  for (uint32_t w = 0; w < kThreads / 32; ++w) {
    const uint4 t = s_tot[w];
    if (w < wrp) { pa += t.x; pb += t.y; }
    sa += t.x; sb += t.y; kt += t.z;
  }
  // a field holds at most 1024 (entries of one j in the tile), so the 16-bit fields never carry
  const uint32_t t0 = sa & 0xFFFFu, t1 = sa >> 16, t2 = sb & 0xFFFFu, t3 = sb >> 16;
  const uint32_t ea = pa + ia - ca, eb = pb + ib - cb;
  uint32_t pos[4] = {ea & 0xFFFFu, t0 + (ea >> 16), t0 + t1 + (eb & 0xFFFFu), t0 + t1 + t2 + (eb >> 16)};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (sel[j]) {
      const uint32_t i0 = (uint32_t)base + (uint32_t)(j * kThreads + tid) * 4u;  // indices fit 32 bits: d < 2^32
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((sel[j] >> k) & 1u) {
          if (pos[j] < kTile) region[pos[j]] = make_uint2(__float_as_uint(compc(v[j], k)), i0 + k);
          ++pos[j];
        }
    }
  }
  if (tid == 0) *info = make_uint4(t0 + t1 + t2 + t3, kt, 0u, 0u);
}

// ---------------------------------------------------------------- pass1
// One CTA per 4096-entry tile: v = source, written over delta; with a predicted band the tile is
// marked while v is still in registers.
template <int SRC, bool FULL>
__device__ __forceinline__ void pass1_tile(const SrcParams& src, uint32_t row, uint64_t base, float* out_row, bool marking,
                                           uint32_t key_lo, uint32_t key_hi, uint2* region, uint4* info, uint4* s_tot) {
  const uint32_t tid = threadIdx.x;
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
  if constexpr (SRC == SRC_WORKER_PLAIN) {
    // v is the gradient itself and stays where it is; nothing is stored and nothing will be zeroed
  } else if constexpr (FULL) {
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
  if (marking) mark_tile<FULL>(v, cnt, base, key_lo, key_hi, SRC == SRC_WORKER_PLAIN ? nullptr : out_row, region, info, s_tot);
}

template <int SRC>
__global__ void __launch_bounds__(kThreads, is_worker_src(SRC) || SRC == SRC_SRV_TOPK ? 5 : kServerCtasPerSm) k_topk_pass1(const SrcParams src, float* v_out, const TopkPred* pred, uint2* list,
                                                         uint64_t cap, uint4* tile_info, uint64_t ntile) {
  pdl_prologue();
  __shared__ uint4 s_tot[kThreads / 32];
  const uint32_t row = blockIdx.y;
  const uint64_t tile = blockIdx.x, base = tile * kTile;
  const uint64_t d = src.d;
  uint32_t key_lo = 1, key_hi = 0;
  const bool marking = predicted_band(pred, row, &key_lo, &key_hi);
  float* out_row = v_out + (uint64_t)row * d;
  uint2* region = list + (uint64_t)row * cap + base;
  uint4* info = tile_info + (uint64_t)row * ntile + tile;
  if (src.vec && base + kTile <= d) {
    pass1_tile<SRC, true>(src, row, base, out_row, marking, key_lo, key_hi, region, info, s_tot);
  } else {
    pass1_tile<SRC, false>(src, row, base, out_row, marking, key_lo, key_hi, region, info, s_tot);
  }
}

// ---------------------------------------------------------------- pick
// Called by all NT threads of a CTA (NT = 1024 or 256).  h: 4096 counters.  Finds the bin where the
// count from the top reaches `want` and how many entries are still to take inside it: s_out[0] = bin,
// s_out[1] = remainder, s_out[2] = total count (valid after the final barrier; s_out[0..1] only if
// 1 <= want <= total).  s_warp: 32 words.
template <int NT = 1024>
__device__ __forceinline__ void cta_pick(const uint32_t* h, uint32_t want, uint32_t* s_warp, uint32_t* s_out) {
  constexpr uint32_t BPT = kBins1 / NT;  // bins per thread
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5;
  // thread t owns bins BPT*(NT-1 - t) .. +BPT-1, so that a forward scan over threads walks bins downwards
  const uint32_t b0 = BPT * ((uint32_t)NT - 1u - tid);
  uint32_t c[BPT];
  uint32_t mine = 0;
#pragma unroll
  for (uint32_t i = 0; i < BPT; ++i) {
    c[i] = h[b0 + i];
    mine += c[i];
  }
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  if (lane == 31) s_warp[wrp] = incl;
  __syncthreads();
  if (wrp == 0) {
    const uint32_t w = lane < (uint32_t)NT / 32u ? s_warp[lane] : 0u;
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= (uint32_t)o) wi += y;
    }
    s_warp[lane] = wi - w;  // exclusive prefix of the warp totals
  }
  __syncthreads();
  const uint32_t above = s_warp[wrp] + incl - mine;  // entries in bins above this thread's own
  if (tid == (uint32_t)NT - 1u) s_out[2] = above + mine;
  if (want > above && want <= above + mine) {
    uint32_t cum = above, tb = b0 + BPT - 1u;
#pragma unroll
    for (int i = (int)BPT - 1; i >= 0; --i) {
      if (want <= cum + c[i]) { tb = b0 + (uint32_t)i; break; }
      cum += c[i];
    }
    s_out[0] = tb;
    s_out[1] = want - cum;
  }
  __syncthreads();
}

// ---------------------------------------------------------------- full histogram (after a miss)
// If pass1 marked with a band that then missed, the entries it zeroed come back first: a tile's
// region holds only entries of that tile, so the CTA that histograms a tile restores it itself.
__global__ void __launch_bounds__(kThreads) k_topk_hist(float* v_io, uint64_t d, int vec, int keep_error, const TopkState* state,
                                                        const TopkPred* pred, const uint2* list, uint64_t cap,
                                                        const uint4* tile_info, uint32_t* hist) {
  pdl_prologue();
  __shared__ uint32_t s_hist[kBins1];
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  if (!state[row].need_full) return;
  for (uint32_t b = tid; b < kBins1; b += kThreads) s_hist[b] = 0;
  uint32_t band_lo = 1, band_hi = 0;
  // what pass1 saw: pred changes only at the end.  Without an error to keep nothing was zeroed.
  const bool marked = predicted_band(pred, row, &band_lo, &band_hi) && keep_error;
  float* vrow = v_io + (uint64_t)row * d;
  const uint64_t ntile = (d + kTile - 1) / kTile;
  for (uint64_t tile = blockIdx.x; tile < ntile; tile += gridDim.x) {
    if (marked) {
      const uint4 info = tile_info[(uint64_t)row * ntile + tile];
      const uint32_t n = min(info.x, (uint32_t)kTile);
      const uint2* region = list + (uint64_t)row * cap + tile * kTile;
      for (uint32_t i = tid; i < n; i += kThreads) {
        const uint2 e = region[i];
        if ((e.x & 0x7fffffffu) > band_hi && (e.y >> 12) == tile && e.y < d) vrow[e.y] = __uint_as_float(e.x);
      }
    }
    __syncthreads();  // restored entries are read below by other threads; also orders s_hist clearing
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

// ---------------------------------------------------------------- tile regions -> dense list
// Exclusive prefix of one value per thread over the CTA (blockDim a multiple of 32, at most 1024).
// s_warp: 33 words.  *total = sum over the CTA.  Ends with a barrier; s_warp may be reused after
// the next barrier the caller passes.
__device__ __forceinline__ uint32_t cta_excl_scan(uint32_t val, uint32_t* s_warp, uint32_t* total) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5, warps = blockDim.x >> 5;
  uint32_t incl = val;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  if (lane == 31) s_warp[wrp] = incl;
  __syncthreads();
  if (wrp == 0) {
    const uint32_t w = lane < warps ? s_warp[lane] : 0u;
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= (uint32_t)o) wi += y;
    }
    s_warp[lane] = wi - w;
    if (lane == 31) s_warp[32] = wi;
  }
  __syncthreads();
  *total = s_warp[32];
  return s_warp[wrp] + incl - val;
}

// One batch of up to 64 region entries, two neighbours per lane (q.x, q.y = first entry, q.z, q.w =
// second): those not above the band (key <= fhi) are the candidates; they go to the dense list as
// (key, index) from slot `run` on, in entry order.
template <bool HIST>
__device__ __forceinline__ void put_candidates(uint4 q, bool valid0, bool valid1, uint32_t fhi, uint32_t& run, uint2* drow,
                                               uint64_t cap, uint32_t* s_hist, uint32_t lane) {
  const uint32_t key0 = q.x & 0x7fffffffu, key1 = q.z & 0x7fffffffu;
  const bool is0 = valid0 && key0 <= fhi, is1 = valid1 && key1 <= fhi;
  const uint32_t b0 = __ballot_sync(0xffffffffu, is0), b1 = __ballot_sync(0xffffffffu, is1);
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t pos = run + __popc(b0 & lt) + __popc(b1 & lt);
  if (is0) {
    if (pos < cap) drow[pos] = make_uint2(key0, q.y);
    if (HIST) atomicAdd(&s_hist[key0 >> 19], 1u);
    ++pos;
  }
  if (is1) {
    if (pos < cap) drow[pos] = make_uint2(key1, q.w);
    if (HIST) atomicAdd(&s_hist[key1 >> 19], 1u);
  }
  run += __popc(b0) + __popc(b1);
}

// The first / a later 64-entry batch of a region of n entries (regions are 16-byte aligned).
__device__ __forceinline__ uint4 region_batch(const uint2* region, uint32_t i0, uint32_t n, uint32_t lane) {
  return i0 + 2u * lane < n ? reinterpret_cast<const uint4*>(region)[(i0 >> 1) + lane] : make_uint4(0u, 0u, 0u, 0u);
}

// Copies the candidates out of the tile regions into one dense list per vector; a tile's
// candidates stay together and in index order, the tiles of a CTA follow one another.  Each CTA
// takes a contiguous run of tiles; the tile_info counts say how many candidates each region
// holds, so one prefix sum per CTA and ONE reservation in the dense list place them all (the
// counters of all vectors share a cache line, and atomics on one line are served one after the
// other).  With HIST the top-12-bit histogram of the keys is counted on the way.  Returns this
// thread's share of the "entries above the band" counts.  s_n, s_off: blockDim words each;
// s_warp: 34 words.  Called by whole CTAs.
template <bool HIST>
__device__ __forceinline__ uint32_t gather_tiles(const uint2* lrow, const uint4* info, uint64_t ntile, uint2* drow,
                                                 uint64_t cap, uint32_t* dense_count, uint32_t fhi, uint32_t* s_hist,
                                                 uint32_t* s_n, uint32_t* s_off, uint32_t* s_warp) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5, nthr = blockDim.x, warps = nthr >> 5;
  const uint64_t per = (ntile + gridDim.x - 1) / gridDim.x;
  const uint64_t c0 = (uint64_t)blockIdx.x * per, c1 = min(ntile, c0 + per);
  uint32_t kept = 0;
  for (uint64_t r0 = c0; r0 < c1; r0 += nthr) {
    uint4 mine = make_uint4(0u, 0u, 0u, 0u);
    if (r0 + tid < c1) mine = info[r0 + tid];
    const uint32_t n = min(mine.x, (uint32_t)kTile), above = min(mine.y, n);
    kept += above;
    uint32_t total;
    const uint32_t excl = cta_excl_scan(n - above, s_warp, &total);
    s_n[tid] = n;
    s_off[tid] = excl;
    if (tid == 0) s_warp[33] = total ? atomicAdd(dense_count, total) : 0u;
    __syncthreads();
    const uint32_t base = s_warp[33];
    const uint32_t ntl = (uint32_t)min((uint64_t)nthr, c1 - r0);
    // a warp takes four tiles at a time and has the first 64 entries of each in flight at once
    for (uint32_t i = wrp; i < ntl; i += 4 * warps) {
      uint32_t nn[4];
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t iu = i + u * warps;
        nn[u] = iu < ntl ? s_n[iu] : 0u;
        q[u] = region_batch(lrow + (r0 + iu) * kTile, 0, nn[u], lane);  // no read where nn[u] == 0
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (nn[u] == 0) continue;
        const uint32_t iu = i + u * warps;
        const uint2* reg = lrow + (r0 + iu) * kTile;
        uint32_t run = base + s_off[iu];
        put_candidates<HIST>(q[u], 2u * lane < nn[u], 2u * lane + 1u < nn[u], fhi, run, drow, cap, s_hist, lane);
        for (uint32_t i0 = 64; i0 < nn[u]; i0 += 64)
          put_candidates<HIST>(region_batch(reg, i0, nn[u], lane), i0 + 2u * lane < nn[u], i0 + 2u * lane + 1u < nn[u], fhi,
                               run, drow, cap, s_hist, lane);
      }
    }
    __syncthreads();  // s_n, s_off and s_warp are rewritten by the next round
  }
  return kept;
}

// ---------------------------------------------------------------- pick + mark + compact (after a miss)
// The rest of the full route in one kernel, for the vectors whose prediction missed.  Every CTA takes
// the level-1 pick for itself from the full histogram k_topk_hist left (4096 counters), rebuilds the
// regions of its run of tiles for that exact bin -- entries in bins above it are kept (and zeroed in
// the residual), entries inside it are the candidates -- and copies its candidates into the dense
// list.  The CTA of a vector that finishes last (a ticket counter, no waiting) records the pick for
// the kernels that follow and clears the histogram.
__global__ void __launch_bounds__(kThreads) k_topk_mark(float* v_io, uint64_t d, int vec, int keep_error, TopkState* state,
                                                        uint2* list, uint64_t cap, uint4* tile_info, uint64_t ntile,
                                                        uint32_t* hist, uint32_t k, uint2* dense, uint32_t* dense_count,
                                                        uint32_t* done) {
  pdl_prologue();
  __shared__ uint4 s_tot[kThreads / 32];
  __shared__ uint32_t s_n[kThreads], s_off[kThreads], s_warp[34], s_out[3];
  __shared__ uint32_t s_last;
  const uint32_t tid = threadIdx.x, row = blockIdx.y;
  TopkState* st = state + row;
  if (!st->need_full) return;
  uint32_t* h = hist + (uint64_t)row * kBins1;
  if (tid == 0) { s_out[0] = 0; s_out[1] = 0; s_out[2] = 0; }
  __syncthreads();
  cta_pick<kThreads>(h, k, s_warp, s_out);
  const uint32_t tb1 = s_out[0], k_rem = s_out[1];
  const uint32_t lo = tb1 << 19, hi = lo | 0x7FFFFu;
  float* vrow = v_io + (uint64_t)row * d;
  // the run of tiles gather_tiles will take for this CTA
  const uint64_t per = (ntile + gridDim.x - 1) / gridDim.x;
  const uint64_t c0 = (uint64_t)blockIdx.x * per, c1 = min(ntile, c0 + per);
  for (uint64_t tile = c0; tile < c1; ++tile) {
    const uint64_t base = tile * kTile;
    const bool full = vec && base + kTile <= d;
    float4 v[4];
    uint32_t cnt[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t e = base + (uint64_t)(j * kThreads + tid) * 4u;
      cnt[j] = e < d ? (uint32_t)min((uint64_t)4, d - e) : 0u;
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cnt[j]) {
        if (vec && cnt[j] == 4) {
          v[j] = *reinterpret_cast<const float4*>(vrow + e);
        } else {
#pragma unroll
          for (int k2 = 0; k2 < 4; ++k2)
            if ((uint32_t)k2 < cnt[j]) comp(v[j], k2) = vrow[e + k2];
        }
      }
    }
    uint2* region = list + (uint64_t)row * cap + base;
    uint4* info = tile_info + (uint64_t)row * ntile + tile;
    float* zero_in = keep_error ? vrow : nullptr;
    if (full) mark_tile<true>(v, cnt, base, lo, hi, zero_in, region, info, s_tot);
    else mark_tile<false>(v, cnt, base, lo, hi, zero_in, region, info, s_tot);
    __syncthreads();  // s_tot is written again for the next tile; the tile's region and counts are visible to the CTA
  }
  gather_tiles<false>(list + (uint64_t)row * cap, tile_info + (uint64_t)row * ntile, ntile, dense + (uint64_t)row * cap, cap,
                      &dense_count[row], hi, nullptr, s_n, s_off, s_warp);
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&done[row], 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  // every CTA of the vector has read the histogram: clear it for the next digit
  for (uint32_t b = tid; b < kBins1; b += kThreads) h[b] = 0;
  if (tid != 0) return;
  done[row] = 0;
  st->tb1 = tb1;
  st->k_rem = k_rem;
  st->zeroed_above = hi;  // mark zeroed the bins above the threshold bin
}

// ---------------------------------------------------------------- list histogram + pick
// One radix digit from the candidate list: LEVEL 1 = key bits 30..19 (and the verdict on the
// prediction), LEVEL 2 = bits 18..7, LEVEL 3 = bits 6..0 (tau and r complete; tau is remembered
// for the next step's prediction).  Several CTAs per vector histogram slices of the list into the
// vector's global histogram; the CTA that finishes last (a ticket counter, no waiting) picks the
// digit and clears histogram and ticket.
template <int LEVEL>
__global__ void __launch_bounds__(1024) k_topk_lhist(const uint2* list, uint64_t cap, const uint4* tile_info, uint64_t ntile,
                                                     uint2* dense, uint32_t* dense_count, uint32_t* kept_count,
                                                     TopkState* state, uint32_t* hist, uint32_t* done, uint32_t k,
                                                     TopkPred* pred, uint32_t* dev_status) {
  pdl_prologue();
  __shared__ uint32_t s_hist[kBins1];
  __shared__ uint32_t s_warp[34], s_out[3];
  __shared__ uint32_t s_last, s_kept;
  constexpr uint32_t NB = LEVEL == 3 ? 128u : 4096u;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  TopkState* st = state + row;
  uint32_t band_lo = 1, band_hi = 0;
  // LEVEL 1 reads what pass1 wrote, which exists only if pass1 had a band to work with
  const bool readable = LEVEL != 1 || predicted_band(pred, row, &band_lo, &band_hi);
  const uint32_t tb1 = st->tb1, top24 = (st->tb1 << 12) | st->tb2;
  for (uint32_t b = tid; b < NB; b += 1024) s_hist[b] = 0;
  if (tid == 0) s_kept = 0;
  __syncthreads();
  if constexpr (LEVEL == 1) {
    __shared__ uint32_t s_n[1024], s_off[1024];
    uint32_t kept = 0;
    if (readable)
      kept = gather_tiles<true>(list + (uint64_t)row * cap, tile_info + (uint64_t)row * ntile, ntile,
                                dense + (uint64_t)row * cap, cap, &dense_count[row], band_hi, s_hist, s_n, s_off, s_warp);
    kept = __reduce_add_sync(0xffffffffu, kept);
    if (lane == 0 && kept) atomicAdd(&s_kept, kept);
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
  __syncthreads();
  uint32_t* h = hist + (uint64_t)row * kBins1;
  for (uint32_t b = tid; b < NB; b += 1024) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&h[b], c);
  }
  if (LEVEL == 1 && tid == 0 && s_kept) atomicAdd(&kept_count[row], s_kept);
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
    const bool hit = readable && want >= 1 && want <= s_out[2];
    atomicAdd(&dev_status[hit ? DS_DEV_WORD_TOPK_PREDICTED : DS_DEV_WORD_TOPK_FULL], 1u);  // one per selection
    if (hit) {
      st->tb1 = s_out[0];
      st->k_rem = s_out[1];
      st->need_full = 0;
      st->zeroed_above = band_hi;
    } else {
      st->need_full = 1;  // hist and mark rebuild the regions and the list for the exact bin
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

// ---------------------------------------------------------------- emit from the tile regions
// A warp per tile.  The region lists, in index order, every entry that can be kept; the scan gave
// the tile its first output slot (and the number of ties before it), so a ballot per 32 entries
// places them.  Entries above `zeroed_above` were zeroed in the residual when they were listed;
// the kept candidates are zeroed here (delta = v - Q[v], Eq. 3).
__global__ void __launch_bounds__(kThreads) k_topk_emit_list(float* v_io, uint64_t d, const TopkState* state, const uint2* list,
                                                             uint64_t cap, const uint4* tile_info, const uint2* tile_pre,
                                                             uint64_t ntile, uint8_t* payload, uint64_t payload_stride,
                                                             uint64_t off_idx, uint64_t off_val, uint32_t k, float* x,
                                                             float gamma, int keep_error, uint32_t* span_off) {
  pdl_prologue();
  const uint32_t tid = threadIdx.x, lane = tid & 31u, row = blockIdx.y;
  const uint64_t tile = (uint64_t)blockIdx.x * (kThreads / 32) + (tid >> 5);
  if (tile >= ntile) return;
  // the first 64 slots of the region are fetched together with the tile's counts (a region always
  // has kTile slots; those past the count are never looked at), so one memory round trip serves both
  const uint2* region = list + (uint64_t)row * cap + tile * kTile;
  uint4 q = reinterpret_cast<const uint4*>(region)[lane];  // 64 entries per trip, two neighbours per lane
  const uint4 info = tile_info[(uint64_t)row * ntile + tile];
  const uint2 pre = tile_pre[(uint64_t)row * ntile + tile];
  const uint32_t n = min(info.x, (uint32_t)kTile);
  const uint32_t tau = state[row].tau, r = state[row].r, zeroed_above = state[row].zeroed_above;
  const bool ties = info.w != 0;  // the tile holds an entry equal to tau
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t ties_before = pre.y;
  uint32_t run = pre.x + min(pre.y, r);
  if (span_off && lane == 0) {
    // where every span of kSparseSpan indices begins in this vector's ascending index list: the table
    // the ordered sum of sparse payloads works from (a span is a whole number of tiles)
    constexpr uint64_t tps = kSparseSpan / kTile;
    const uint64_t nspan = (ntile + tps - 1) / tps;
    uint32_t* o = span_off + (uint64_t)row * (nspan + 1);
    if (tile % tps == 0) o[tile / tps] = run;
    if (tile == 0) o[nspan] = k;
  }
  if (n == 0) return;
  float* vrow = v_io + (uint64_t)row * d;
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(payload + (uint64_t)row * payload_stride + off_idx);
  float* out_val = reinterpret_cast<float*>(payload + (uint64_t)row * payload_stride + off_val);
  for (uint32_t i0 = 0; i0 < n; i0 += 64) {
    const uint4 q_next = region_batch(region, i0 + 64, n, lane);
    const bool valid0 = i0 + 2u * lane < n, valid1 = i0 + 2u * lane + 1u < n;
    const uint32_t key0 = q.x & 0x7fffffffu, key1 = q.z & 0x7fffffffu;
    bool sel0 = valid0 && key0 > tau, sel1 = valid1 && key1 > tau;
    if (ties) {
      // ties are kept lowest index first until r of them are in
      const bool tie0 = valid0 && key0 == tau, tie1 = valid1 && key1 == tau;
      const uint32_t b0 = __ballot_sync(0xffffffffu, tie0), b1 = __ballot_sync(0xffffffffu, tie1);
      const uint32_t before = ties_before + __popc(b0 & lt) + __popc(b1 & lt);
      if (tie0 && before < r) sel0 = true;
      if (tie1 && before + (tie0 ? 1u : 0u) < r) sel1 = true;
      ties_before += __popc(b0) + __popc(b1);
    }
    const uint32_t s0 = __ballot_sync(0xffffffffu, sel0), s1 = __ballot_sync(0xffffffffu, sel1);
    uint32_t pos = run + __popc(s0 & lt) + __popc(s1 & lt);
    if (sel0) {
      const uint32_t j = q.y;
      const float val = __uint_as_float(q.x);
      if (pos < k) { out_idx[pos] = j; out_val[pos] = val; }  // pos < k whenever the counts are consistent
      if (j < d) {
        if (keep_error && key0 <= zeroed_above) vrow[j] = 0.f;
        if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, val));
      }
      ++pos;
    }
    if (sel1) {
      const uint32_t j = q.w;
      const float val = __uint_as_float(q.z);
      if (pos < k) { out_idx[pos] = j; out_val[pos] = val; }
      if (j < d) {
        if (keep_error && key1 <= zeroed_above) vrow[j] = 0.f;
        if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, val));
      }
    }
    run += __popc(s0) + __popc(s1);
    q = q_next;
  }
}

// ================================================================ pipeline without a list

// pass1 with the full 4096-bin histogram and no marking.
template <int SRC>
__global__ void __launch_bounds__(kThreads) k_topk_pass1_basic(const SrcParams src, float* v_out, uint32_t* hist,
                                                               uint64_t span) {
  pdl_prologue();
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
  pdl_prologue();
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
  pdl_prologue();
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
  pdl_prologue();
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
  pdl_prologue();
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

// Exclusive prefix of the per-segment counts of one vector (in place), or with TILES of the
// per-tile counts in tile_info (written to seg_cnt); checks that exactly k entries will be emitted.
// Called by all 1024 threads of a CTA.
template <bool TILES>
__device__ __forceinline__ void cta_scan_counts(uint32_t row, uint2* seg_cnt, const uint4* tile_info, uint64_t nseg,
                                                TopkState* state, uint32_t k, uint32_t* dev_status) {
  // A round takes 4096 counts: loaded and stored with neighbouring threads on neighbouring counts,
  // scanned with four consecutive counts per thread; shared memory turns one order into the other.
  constexpr int ITEMS = 4;
  __shared__ uint2 s_item[1024 * ITEMS];
  __shared__ uint2 s_warp[32];
  __shared__ uint2 s_carry;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, wrp = tid >> 5;
  uint2* c = seg_cnt + (uint64_t)row * nseg;
  if (tid == 0) s_carry = make_uint2(0, 0);
  for (uint64_t base = 0; base < nseg; base += 1024 * ITEMS) {
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
      const uint64_t i = base + (uint64_t)u * 1024 + tid;
      uint2 item = make_uint2(0, 0);
      if (i < nseg) {
        if (TILES) {
          const uint4 t = __ldcg(&tile_info[(uint64_t)row * nseg + i]);   // other CTAs counted into it just now
          item = make_uint2(t.y + t.z, t.w);  // above the band + candidates above tau; candidates equal to tau
        } else {
          item = c[i];
        }
      }
      s_item[u * 1024 + tid] = item;
    }
    __syncthreads();
    uint2 mine[ITEMS];
    uint2 sum = make_uint2(0, 0);
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
      mine[u] = s_item[tid * ITEMS + u];
      sum.x += mine[u].x;
      sum.y += mine[u].y;
    }
    uint2 incl = sum;
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
    uint2 excl = make_uint2(carry.x + s_warp[wrp].x + incl.x - sum.x, carry.y + s_warp[wrp].y + incl.y - sum.y);
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
      s_item[tid * ITEMS + u] = excl;
      excl.x += mine[u].x;
      excl.y += mine[u].y;
    }
    __syncthreads();
    if (tid == 1023) s_carry = excl;  // the prefix after this round's last count
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
      const uint64_t i = base + (uint64_t)u * 1024 + tid;
      if (i < nseg) c[i] = s_item[u * 1024 + tid];
    }
    __syncthreads();
  }
  __syncthreads();
  if (tid == 0) {
    const uint2 tot = s_carry;
    const uint32_t r = state[row].r;
    state[row].total_gt = tot.x;
    state[row].total_tie = tot.y;
    if (k != 0xFFFFFFFFu && tot.x + min(tot.y, r) != k) atomicOr(dev_status, DS_DEV_TOPK_INCONSISTENT);
  }
}

// Pipeline without a list: the prefix over the segment counts, one CTA per vector.
__global__ void __launch_bounds__(1024) k_topk_scan(uint2* seg_cnt, uint64_t nseg, TopkState* state, uint32_t k,
                                                    uint32_t* dev_status) {
  pdl_prologue();
  cta_scan_counts<false>(blockIdx.x, seg_cnt, nullptr, nseg, state, k, dev_status);
}

// ================================================================ a slice of a vector that lives on several GPUs
// The selection over a vector whose slices sit on different GPUs is the pipeline without a list, cut
// where a histogram is complete: the caller adds the slices' histograms up (an all-reduce of 16 KB) and
// hands the sum back, every slice then picks the same digit.  See ds_server_topk_slice_* in dsq.h.

// The prefix over the segment counts of ONE slice; how many entries the slice holds above tau and equal
// to it, and the tie quota r of the whole vector, go to out[0..2].  No check against k: that is the
// whole vector's business.
__global__ void __launch_bounds__(1024) k_topk_slice_scan(uint2* seg_cnt, uint64_t nseg, TopkState* state, uint32_t* out) {
  pdl_prologue();
  __shared__ uint32_t s_ignore;
  cta_scan_counts<false>(0, seg_cnt, nullptr, nseg, state, 0xFFFFFFFFu, &s_ignore);
  __syncthreads();
  if (threadIdx.x == 0) {
    out[0] = state[0].total_gt;
    out[1] = state[0].total_tie;
    out[2] = state[0].r;
    out[3] = state[0].tau;
  }
}

// The slice's share of the tie quota, decided by the caller from all slices' tie counts.
__global__ void k_topk_slice_quota(TopkState* state, uint32_t ties_to_keep) {
  pdl_prologue();
  if (threadIdx.x == 0 && blockIdx.x == 0) state[0].r = ties_to_keep;
}

// ---------------------------------------------------------------- classify + prefix
// Per tile, how many of its candidates lie above tau (z) and how many equal it (w): the counters
// pass1 / mark left at zero beside the tile's counts.  A tile's candidates are neighbours in the
// dense list, so the lanes of a warp that count for the same counter send one atomic between
// them.  Integer atomics: order-free.  The CTA of a vector that finishes last (a ticket counter, no
// waiting) then takes the exclusive prefix over the vector's tiles, which saves a launch.
__global__ void __launch_bounds__(1024) k_topk_classify(const uint2* dense, const uint32_t* dense_count, uint64_t cap,
                                                        TopkState* state, uint4* tile_info, uint2* tile_pre, uint64_t ntile,
                                                        uint32_t* done, uint32_t k, uint32_t* dev_status) {
  pdl_prologue();
  __shared__ uint32_t s_last;
  const uint32_t row = blockIdx.y, tid = threadIdx.x, lane = tid & 31u;
  const uint2* drow = dense + (uint64_t)row * cap;
  const uint64_t n = min((uint64_t)dense_count[row], cap);
  const uint32_t tau = state[row].tau;
  uint32_t* counters = reinterpret_cast<uint32_t*>(tile_info + (uint64_t)row * ntile);
  const uint64_t step = (uint64_t)gridDim.x * 1024 * 4;
  // the loop bound is the same for all lanes of a warp (i0 - threadIdx.x is), as match needs
  for (uint64_t c0 = (uint64_t)blockIdx.x * 1024 * 4; c0 < n; c0 += step) {
    const uint64_t i0 = c0 + tid;
    uint2 e[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t i = i0 + (uint64_t)u * 1024;
      e[u] = i < n ? drow[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t t = e[u].y >> 12;
      const bool live = i0 + (uint64_t)u * 1024 < n && t < ntile && e[u].x >= tau;
      // word index of the counter inside the vector's tile_info: .z for "above", .w for "equal"
      const uint32_t word = live ? (uint32_t)t * 4u + (e[u].x > tau ? 2u : 3u) : 0xFFFFFFFFu;
      const uint32_t peers = __match_any_sync(0xffffffffu, word);
      if (live && lane == (uint32_t)__ffs(peers) - 1u) atomicAdd(&counters[word], (uint32_t)__popc(peers));
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&done[row], 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) done[row] = 0;
  cta_scan_counts<true>(row, tile_pre, tile_info, ntile, state, k, dev_status);
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
                                                        uint32_t k, float* x, float gamma, uint32_t idx_base) {
  pdl_prologue();
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
          if (pos < k) { out_idx[pos] = (uint32_t)j + idx_base; out_val[pos] = v0[i]; }  // pos < k whenever the counts are consistent
          vrow[j] = 0.f;                                                      // delta = v - Q[v] at a kept entry
          if (x) x[j] = __fsub_rn(x[j], __fmul_rn(gamma, v0[i]));
          ++pos;
        }
        if (b1[i] < 32u) {
          const uint64_t j = (widx + i) * 32u + b1[i];
          if (pos < k) { out_idx[pos] = (uint32_t)j + idx_base; out_val[pos] = v1[i]; }
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
        if (pos < k) { out_idx[pos] = (uint32_t)j + idx_base; out_val[pos] = val; }
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
  // the bitmaps serve the pipeline without a list only; with a list the prefix runs over tiles
  p->off_bm_gt = pos;      pos = round16(pos + (with_list ? 0 : (uint64_t)rows * p->bm_stride * 4));
  p->off_bm_eq = pos;      pos = round16(pos + (with_list ? 0 : (uint64_t)rows * p->bm_stride * 4));
  p->off_seg = pos;        pos = round16(pos + (uint64_t)rows * (with_list ? p->ntile : p->nseg) * sizeof(uint2));
  p->off_list = pos;       pos = round16(pos + (uint64_t)rows * p->list_cap * sizeof(uint2));
  p->off_tile_info = pos;  pos = round16(pos + (with_list ? (uint64_t)rows * p->ntile * sizeof(uint4) : 0));
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
  uint4* tile_info = reinterpret_cast<uint4*>(ws + pl.off_tile_info);
  uint2* dense = reinterpret_cast<uint2*>(ws + pl.off_dense);
  const uint64_t d = src.d, cap = pl.list_cap;
  const uint64_t padded = pl.nseg * (uint64_t)kSegElems;
  uint32_t* done = list_count + rows;        // ticket counters of the list histograms
  uint32_t* kept_count = list_count + 2 * rows;  // entries above the predicted band
  cudaError_t e = cudaMemsetAsync(hist, 0, (uint64_t)rows * kBins1 * 4 + (uint64_t)rows * 12, st);
  if (e != cudaSuccess) return e;

  dim3 g1((unsigned)pl.ntile, rows, 1);  // pass1 with a list: one CTA per tile
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
  uint64_t stride_ctas = rows >= 8 ? 148ull : 148ull * 4ull;
  if (stride_ctas > pl.ntile) stride_ctas = pl.ntile;
  dim3 gm((unsigned)stride_ctas, rows, 1);
  const uint64_t off_val = (uint64_t)(reinterpret_cast<uint8_t*>(io.val) - reinterpret_cast<uint8_t*>(io.idx));

  if (list && k) {
    TopkPred* pred = pl.pred;
#define DSQ_P1(S) launch_pdl(k_topk_pass1<S>, g1, kThreads, st, src, io.v_inout, pred, list, cap, tile_info, pl.ntile)
    DSQ_SWITCH_SRC(srck, DSQ_P1)
#undef DSQ_P1
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // level 1 keeps a whole SM per CTA (registers), so its grid is one wave; levels 2 and 3 fit two per SM
    dim3 gl1((unsigned)(148ull / rows ? 148ull / rows : 1), rows, 1);
    dim3 gl((unsigned)(148ull * 2ull / rows ? 148ull * 2ull / rows : 1), rows, 1);
    launch_pdl(k_topk_lhist<1>, gl1, 1024, st, list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred, io.dev_status);
    launch_pdl(k_topk_hist, gm, kThreads, st, io.v_inout, d, src.vec, io.keep_error, state, pred, list, cap, tile_info, hist);
    launch_pdl(k_topk_mark, gm, kThreads, st, io.v_inout, d, src.vec, io.keep_error, state, list, cap, tile_info, pl.ntile, hist, k32,
               dense, list_count, done);
    launch_pdl(k_topk_lhist<2>, gl, 1024, st, list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred, io.dev_status);
    launch_pdl(k_topk_lhist<3>, gl, 1024, st, list, cap, tile_info, pl.ntile, dense, list_count, kept_count, state, hist, done,
                                         k32, pred, io.dev_status);
    dim3 gc((unsigned)(148ull / rows ? 148ull / rows : 1), rows, 1);   // one wave of 1024-thread CTAs
    launch_pdl(k_topk_classify, gc, 1024, st, dense, list_count, cap, state, tile_info, seg, pl.ntile, done, k32, io.dev_status);
    dim3 ge((unsigned)((pl.ntile + kThreads / 32 - 1) / (kThreads / 32)), rows, 1);
    launch_pdl(k_topk_emit_list, ge, kThreads, st, io.v_inout, d, state, list, cap, tile_info, seg, pl.ntile,
                                              reinterpret_cast<uint8_t*>(io.idx), io.payload_stride, 0, off_val, k32, io.x,
                                              io.gamma, io.keep_error, io.span_off);
    count_launches(8);
    return cudaGetLastError();
  } else {
#define DSQ_P1(S) launch_pdl(k_topk_pass1_basic<S>, g1b, kThreads, st, src, io.v_inout, hist, span)
    DSQ_SWITCH_SRC(srck, DSQ_P1)
#undef DSQ_P1
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (k == 0) return cudaSuccess;  // nothing kept: Q[v] = 0, delta = v, x unchanged
    launch_pdl(k_topk_pick_basic, rows, 1024, st, hist, state, 1, k32);
    launch_pdl(k_topk_mark_basic, gm, kThreads, st, io.v_inout, d, src.vec, state, bm_gt, bm_eq, pl.bm_stride, padded);
    launch_pdl(k_topk_refine<2>, gs, kThreads, st, io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    launch_pdl(k_topk_pick_basic, rows, 1024, st, hist, state, 2, k32);
    launch_pdl(k_topk_refine<3>, gs, kThreads, st, io.v_inout, d, state, bm_eq, pl.bm_stride, hist);
    launch_pdl(k_topk_pick_basic, rows, 1024, st, hist, state, 3, k32);
    launch_pdl(k_topk_finalize, gs, kThreads, st, io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg);
    count_launches(7);
  }
  launch_pdl(k_topk_scan, rows, 1024, st, seg, pl.nseg, state, k32, io.dev_status);
  launch_pdl(k_topk_emit, gs, kThreads, st, io.v_inout, d, state, bm_gt, bm_eq, pl.bm_stride, seg, pl.nseg,
                                       reinterpret_cast<uint8_t*>(io.idx), io.payload_stride, 0, off_val, k32, io.x, io.gamma, 0u);
  count_launches(2);
  return cudaGetLastError();
}


// ---------------------------------------------------------------- stages of the selection over a slice
namespace {
struct SlicePtrs {
  uint32_t* hist;
  TopkState* state;
  uint32_t *bm_gt, *bm_eq;
  uint2* seg;
  TopkPlan pl;
  uint64_t padded;
};
SlicePtrs slice_ptrs(uint64_t d_slice, uint64_t k, void* workspace) {
  SlicePtrs p;
  topk_plan(d_slice, 1, k, false, &p.pl);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.hist = reinterpret_cast<uint32_t*>(ws + p.pl.off_hist);
  p.state = reinterpret_cast<TopkState*>(ws + p.pl.off_state);
  p.bm_gt = reinterpret_cast<uint32_t*>(ws + p.pl.off_bm_gt);
  p.bm_eq = reinterpret_cast<uint32_t*>(ws + p.pl.off_bm_eq);
  p.seg = reinterpret_cast<uint2*>(ws + p.pl.off_seg);
  p.padded = p.pl.nseg * (uint64_t)kSegElems;
  return p;
}
dim3 stride_grid(const TopkPlan& pl) {
  uint64_t ctas = 148ull * 4ull;
  if (ctas > pl.ntile) ctas = pl.ntile;
  return dim3((unsigned)ctas, 1, 1);
}
}  // namespace

uint64_t topk_slice_workspace_bytes(uint64_t d_slice, uint64_t k) {
  TopkPlan pl;
  topk_plan(d_slice, 1, k, false, &pl);
  return pl.bytes;
}

cudaError_t launch_topk_slice_begin(int srck, const SrcParams& src, void* workspace, float* v_out, uint64_t k, uint32_t* hist_out,
                                    cudaStream_t st) {
  const SlicePtrs p = slice_ptrs(src.d, k, workspace);
  cudaError_t e = cudaMemsetAsync(hist_out, 0, kBins1 * 4, st);
  if (e != cudaSuccess) return e;
  uint64_t span = 16 * kTile;
  while (span > kTile && ((p.padded + span - 1) / span) < 148ull * 16ull) span /= 2;
  dim3 g1b((unsigned)((p.padded + span - 1) / span), 1, 1);
#define DSQ_P1(S) launch_pdl(k_topk_pass1_basic<S>, g1b, kThreads, st, src, v_out, hist_out, span)
  DSQ_SWITCH_SRC(srck, DSQ_P1)
#undef DSQ_P1
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_topk_slice_digit(int level, void* workspace, const float* v, uint64_t d_slice, int vec, uint64_t k,
                                    uint32_t* hist_sum, uint32_t* hist_next, cudaStream_t st) {
  const SlicePtrs p = slice_ptrs(d_slice, k, workspace);
  const uint32_t k32 = (uint32_t)k;
  dim3 gs((unsigned)p.pl.nseg, 1, 1);
  cudaError_t e = cudaMemsetAsync(hist_next, 0, kBins1 * 4, st);
  if (e != cudaSuccess) return e;
  launch_pdl(k_topk_pick_basic, 1, 1024, st, hist_sum, p.state, (uint32_t)level, k32);   // clears hist_sum
  if (level == 1) {
    launch_pdl(k_topk_mark_basic, stride_grid(p.pl), kThreads, st, v, d_slice, vec, p.state, p.bm_gt, p.bm_eq, p.pl.bm_stride, p.padded);
    launch_pdl(k_topk_refine<2>, gs, kThreads, st, v, d_slice, p.state, p.bm_eq, p.pl.bm_stride, hist_next);
    count_launches(3);
  } else if (level == 2) {
    launch_pdl(k_topk_refine<3>, gs, kThreads, st, v, d_slice, p.state, p.bm_eq, p.pl.bm_stride, hist_next);
    count_launches(2);
  } else {
    launch_pdl(k_topk_finalize, gs, kThreads, st, v, d_slice, p.state, p.bm_gt, p.bm_eq, p.pl.bm_stride, p.seg, p.pl.nseg);
    launch_pdl(k_topk_slice_scan, 1, 1024, st, p.seg, p.pl.nseg, p.state, hist_next);
    count_launches(3);
  }
  return cudaGetLastError();
}

cudaError_t launch_topk_slice_emit(void* workspace, float* v_io, uint64_t d_slice, uint64_t k, uint32_t ties_to_keep, uint32_t count,
                                   uint32_t idx_base, uint32_t* out_idx, float* out_val, float* x, float gamma, cudaStream_t st) {
  const SlicePtrs p = slice_ptrs(d_slice, k, workspace);
  dim3 gs((unsigned)p.pl.nseg, 1, 1);
  const uint64_t off_val = (uint64_t)(reinterpret_cast<uint8_t*>(out_val) - reinterpret_cast<uint8_t*>(out_idx));
  launch_pdl(k_topk_slice_quota, 1, 32, st, p.state, ties_to_keep);
  launch_pdl(k_topk_emit, gs, kThreads, st, v_io, d_slice, p.state, p.bm_gt, p.bm_eq, p.pl.bm_stride, p.seg, p.pl.nseg,
             reinterpret_cast<uint8_t*>(out_idx), (uint64_t)0, (uint64_t)0, off_val, count, x, gamma, idx_base);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace dsq
