/*
 * DoubleSqueeze oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of what one DoubleSqueeze
 * iteration computes (Algorithm 1; Section 3.1, Eq. 2-4; the compression
 * options of Section 3.2 and of the "Implementations and setups" paragraph of
 * Section 5.1).  It exists so that the CUDA library can be checked against
 * something written directly from the paper.  It shares no code, header,
 * table or constant generator with the CUDA path and must never be called
 * from it; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.
 *
 * Arithmetic model.  Every state array is IEEE-754 binary32.  Every
 * elementwise operation below is a single round-to-nearest-even binary32
 * operation, written one per statement; the file is compiled with
 * -ffp-contract=off so no multiply-add is fused.  A chunk reduction is
 * PAIRWISE (cascade) SUMMATION in binary32 over the chunk in index order,
 * the chunk being padded with +0 up to its nominal power-of-two length:
 *     S(a[lo,hi)) = S(a[lo,mid)) + S(a[mid,hi)),  mid = (lo+hi)/2,  S(a[i]) = a[i].
 * That fixes the rounding order, so a quantised code that depends on a chunk
 * norm is decided in one well-defined precision.
 *
 * Parity pins (tests/test_oracle_*.py): identity => parallel SGD bitwise;
 * C + delta_new == g + delta_old; the telescoping identity of Section 3.3
 * (Eq. 5-6); sign scale == ||v||_1/len (or ||v||_2/sqrt(len)) and its closed-form residual energy;
 * top-k against a brute-force stable sort; QSGD unbiasedness and variance by
 * Monte Carlo plus its deterministic special cases; clipping against worked
 * binary cases, its error bound and idempotence; randomised sparsification by
 * its keep frequency, its mean, and the structure of what it sends; Philox4x32-10 against an
 * independent library implementation; pairwise summation against hand-derived
 * rounding cases; the ternary quantiser by Monte Carlo (unbiased before its
 * scaling), its always-kept largest entry and its l1 factor; the passes without
 * compensation against plain compressed SGD.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG -1
#define ORC_ERR_NOMEM -2

/* ------------------------------------------------------------------------ */
/* helpers                                                                  */
/* ------------------------------------------------------------------------ */

static uint32_t f32_bits(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  return u;
}

static int is_pow2_u32(uint32_t x) { return x != 0 && (x & (x - 1)) == 0; }

/* Pairwise summation of a[0..len), len a power of two (see file header). */
static float pairwise_sum(const float* a, size_t len) {
  if (len == 1) return a[0];
  size_t half = len / 2;
  float left = pairwise_sum(a, half);
  float right = pairwise_sum(a + half, half);
  float s = left + right;
  return s;
}

/* The same sum over a[0..len) padded with +0 up to L entries (L a power of two, len <= L), without
 * storing the padding: a half that holds only padding sums to +0, and x + (+0) = x for every x that
 * can occur here (the terms are |v| or v*v, never -0). */
static float pairwise_sum_padded(const float* a, uint64_t len, uint64_t L) {
  if (len == 0) return 0.0f;
  if (L == 1) return a[0];
  uint64_t half = L / 2;
  float left = pairwise_sum_padded(a, len < half ? len : half, half);
  float right = pairwise_sum_padded(a + half, len > half ? len - half : 0, half);
  float s = left + right;
  return s;
}

static uint64_t next_pow2_u64(uint64_t x) {
  uint64_t p = 1;
  while (p < x) p <<= 1;
  return p;
}

float orc_pairwise_sum_padded(const float* a, uint64_t len, uint64_t L) {
  if (L == 0 || (L & (L - 1)) != 0 || len > L) return NAN;
  return pairwise_sum_padded(a, len, L);
}

/* Exposed for the tests that pin the summation order. */
float orc_pairwise_sum(const float* a, uint64_t len) {
  if (len == 0 || (len & (len - 1)) != 0) return NAN;
  return pairwise_sum(a, (size_t)len);
}

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11): the counter-based generator that supplies the   */
/* randomness omega of a randomised Q (footnote to Section 1).               */
/* ------------------------------------------------------------------------ */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t mult0 = 0xD2511F53u; /* multiplier applied to word 0 */
  const uint64_t mult1 = 0xCD9E8D57u; /* multiplier applied to word 2 */
  const uint32_t weyl0 = 0x9E3779B9u; /* key schedule increments */
  const uint32_t weyl1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = mult0 * (uint64_t)c0;
    uint64_t p1 = mult1 * (uint64_t)c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += weyl0;
    k1 += weyl1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------------------------------------ */
/* Elementwise steps of Algorithm 1                                          */
/* ------------------------------------------------------------------------ */

/* Eq. 2: error-compensated gradient  v = g + delta. */
void orc_ef_add(const float* g, const float* delta, uint64_t d, float* v) {
  for (uint64_t j = 0; j < d; ++j) {
    float s = g[j] + delta[j];
    v[j] = s;
  }
}

/* Eq. 3 and the second line of Eq. 4: residual  delta = v - Q[v]. */
void orc_residual(const float* v, const float* C, uint64_t d, float* delta) {
  for (uint64_t j = 0; j < d; ++j) {
    float r = v[j] - C[j];
    delta[j] = r;
  }
}

/* First line of Eq. 4:  v = delta_s + (1/n) sum_i Q[v_i].
 * The sum runs over workers in order i = 0..n-1 starting from +0, is scaled
 * by inv_n = 1/n rounded once, then delta_s is added.  C_all is [n, d]. */
void orc_server_mean_add(const float* C_all, uint32_t n, uint64_t d, const float* delta_s, float* v) {
  float one = 1.0f;
  float inv_n = one / (float)n;
  for (uint64_t j = 0; j < d; ++j) {
    float acc = 0.0f;
    for (uint32_t i = 0; i < n; ++i) {
      float t = acc + C_all[(uint64_t)i * d + j];
      acc = t;
    }
    float mean = acc * inv_n;
    float s = mean + delta_s[j];
    v[j] = s;
  }
}

/* Model update of Algorithm 1:  x = x - gamma * Q[v]  (two roundings). */
void orc_apply_update(float* x, const float* C, float gamma, uint64_t d) {
  for (uint64_t j = 0; j < d; ++j) {
    float t = gamma * C[j];
    float r = x[j] - t;
    x[j] = r;
  }
}

/* ------------------------------------------------------------------------ */
/* Q = identity: Algorithm 1 then is plain parallel SGD (Section 1).         */
/* ------------------------------------------------------------------------ */

int orc_q_identity(const float* v, uint64_t d, float* C) {
  for (uint64_t j = 0; j < d; ++j) C[j] = v[j];
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Q = 1-bit quantisation with a scaling factor (Section 3.2 "1-Bit          */
/* Quantization"; Section 5.1 "1-bit compression": the factor is magnitude   */
/* of the compensated gradient over magnitude of the sign vector).  The      */
/* factor is taken per chunk of L consecutive elements of the flat vector,   */
/* len_c being the true length of the (possibly short, last) chunk.          */
/*   norm = 1: magnitude = l1 norm, factor = ||v_c||_1 / len_c               */
/*   norm = 2: magnitude = l2 norm (the norm Section 3.2 prints),            */
/*             factor = ||v_c||_2 / sqrt(len_c)                              */
/* A zero has no sign to send, so bit = (v >= 0).                            */
/*   bits : ceil(d/32) words, element j -> bit (j%32) of word j/32, pad 0    */
/*   scale: ceil(d/L) floats                                                 */
/*   C    : d floats (may be NULL)                                           */
/* ------------------------------------------------------------------------ */

static int q_sign1_whole(const float* v, uint64_t d, uint32_t norm, uint32_t* bits, float* scale, float* C);

int orc_q_sign1(const float* v, uint64_t d, uint32_t L, uint32_t norm, uint32_t* bits, float* scale, float* C) {
  if (norm != 1 && norm != 2) return ORC_ERR_ARG;
  if (L == 0) return q_sign1_whole(v, d, norm, bits, scale, C);
  if (!is_pow2_u32(L)) return ORC_ERR_ARG;
  uint64_t nw = (d + 31) / 32, nc = (d + L - 1) / L;
  float* term = (float*)malloc(sizeof(float) * L);
  if (!term) return ORC_ERR_NOMEM;
  memset(bits, 0, sizeof(uint32_t) * nw);
  for (uint64_t c = 0; c < nc; ++c) {
    uint64_t lo = c * L, hi = lo + L < d ? lo + L : d;
    uint32_t len = (uint32_t)(hi - lo);
    float s;
    if (norm == 1) {
      for (uint32_t t = 0; t < L; ++t) term[t] = t < len ? fabsf(v[lo + t]) : 0.0f;
      float l1 = pairwise_sum(term, L);
      s = l1 / (float)len;
    } else {
      for (uint32_t t = 0; t < L; ++t) {
        float e = t < len ? v[lo + t] : 0.0f;
        float e2 = e * e;
        term[t] = e2;
      }
      float ss = pairwise_sum(term, L);
      float l2 = sqrtf(ss);
      float root_len = sqrtf((float)len);
      s = l2 / root_len;
    }
    scale[c] = s;
    for (uint64_t j = lo; j < hi; ++j) {
      int nonneg = v[j] >= 0.0f;
      if (nonneg) bits[j / 32] |= (uint32_t)1 << (j % 32);
      if (C) C[j] = nonneg ? s : -s;
    }
  }
  free(term);
  return ORC_OK;
}

/* L = 0: the operator exactly as Section 3.2 and Section 5.1 state it, with ONE scaling factor for the
 * whole vector: magnitude of v over magnitude of sign(v), i.e. ||v||_1 / d (norm = 1) or
 * ||v||_2 / sqrt(d) (norm = 2).  The sum runs pairwise over the vector padded with +0 to the next
 * power of two.  scale holds one float. */
static int q_sign1_whole(const float* v, uint64_t d, uint32_t norm, uint32_t* bits, float* scale, float* C) {
  uint64_t nw = (d + 31) / 32;
  float* term = (float*)malloc(sizeof(float) * (d ? d : 1));
  if (!term) return ORC_ERR_NOMEM;
  memset(bits, 0, sizeof(uint32_t) * nw);
  float s;
  if (norm == 1) {
    for (uint64_t j = 0; j < d; ++j) term[j] = fabsf(v[j]);
    float l1 = pairwise_sum_padded(term, d, next_pow2_u64(d));
    s = l1 / (float)d;
  } else {
    for (uint64_t j = 0; j < d; ++j) {
      float e2 = v[j] * v[j];
      term[j] = e2;
    }
    float ss = pairwise_sum_padded(term, d, next_pow2_u64(d));
    float l2 = sqrtf(ss);
    float root_d = sqrtf((float)d);
    s = l2 / root_d;
  }
  scale[0] = s;
  for (uint64_t j = 0; j < d; ++j) {
    int nonneg = v[j] >= 0.0f;
    if (nonneg) bits[j / 32] |= (uint32_t)1 << (j % 32);
    if (C) C[j] = nonneg ? s : -s;
  }
  free(term);
  return ORC_OK;
}

int orc_decode_sign1(const uint32_t* bits, const float* scale, uint64_t d, uint32_t L, float* C) {
  for (uint64_t j = 0; j < d; ++j) {
    float s = L ? scale[j / L] : scale[0];
    int nonneg = (bits[j / 32] >> (j % 32)) & 1u;
    C[j] = nonneg ? s : -s;
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Q = clipping (the "Clipping" option of Section 3.2: the low-order bits of  */
/* every number are dropped; deterministic, biased).  Reading: the number is */
/* its binary32 word and its low b bits are cleared, which keeps the sign,   */
/* exponent and the leading 23 - b fraction bits (b <= 23), i.e. truncates   */
/* the magnitude toward zero.  What is sent per entry is the surviving high  */
/* 32 - b bits; b is 16 or 24 so that an entry is a 16- or an 8-bit word.    */
/*   hi : d words of (32 - b) bits, little-endian bytes                      */
/*   C  : d floats (may be NULL)                                             */
/* ------------------------------------------------------------------------ */

int orc_q_clip(const float* v, uint64_t d, uint32_t b, uint8_t* hi, float* C) {
  if (b != 16 && b != 24) return ORC_ERR_ARG;
  uint32_t bytes = (32 - b) / 8;
  for (uint64_t j = 0; j < d; ++j) {
    uint32_t u = f32_bits(v[j]);
    uint32_t kept = u >> b;       /* the high 32 - b bits */
    uint32_t cleared = kept << b; /* the number with its low b bits set to zero */
    for (uint32_t t = 0; t < bytes; ++t) hi[j * bytes + t] = (uint8_t)(kept >> (8 * t));
    if (C) memcpy(&C[j], &cleared, sizeof cleared);
  }
  return ORC_OK;
}

int orc_decode_clip(const uint8_t* hi, uint64_t d, uint32_t b, float* C) {
  if (b != 16 && b != 24) return ORC_ERR_ARG;
  uint32_t bytes = (32 - b) / 8;
  for (uint64_t j = 0; j < d; ++j) {
    uint32_t kept = 0;
    for (uint32_t t = 0; t < bytes; ++t) kept |= (uint32_t)hi[j * bytes + t] << (8 * t);
    uint32_t u = kept << b;
    memcpy(&C[j], &u, sizeof u);
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Q = randomised sparsification (the last option of Section 3.2: a number   */
/* survives with probability p, scaled by 1/p so that the operator is        */
/* unbiased, else it becomes 0).  Reading: p = 1/S with S a power of two,    */
/* and the numbers of a chunk of L consecutive elements share one random     */
/* draw (systematic sampling): with o uniform in {0, ..., S-1}, the element  */
/* at offset t in the chunk survives iff t mod S == o.  Every element still  */
/* survives with probability exactly 1/S, which is all the option states,    */
/* and every chunk sends exactly L/S values whose positions follow from o.   */
/* The draw is the first output word of Philox4x32-10 with key = seed and    */
/* counter = (0xFFFFFFFF, chunk, wid, step), reduced mod S.                  */
/*   scaled = 1: survivors become S * v (exact, a power of two): the option  */
/*               as printed.  Unbiased, but E||v - Q[v]||^2 = (S-1)||v||^2,  */
/*               no contraction: the compensated error grows under it.       */
/*   scaled = 0: survivors keep v: E||v - Q[v]||^2 = (1 - 1/S)||v||^2, a     */
/*               contraction, the form error compensation can carry.         */
/*   val : ceil(d/L) * (L/S) floats; slot j/S holds Q[v]_j of the survivor   */
/*         j, slots of positions past d stay +0                              */
/*   off : ceil(d/L) words, the o of every chunk                             */
/*   C   : d floats (may be NULL)                                            */
/* ------------------------------------------------------------------------ */

int orc_q_rsparse(const float* v, uint64_t d, uint32_t L, uint32_t S, uint32_t scaled, uint64_t seed, uint32_t step,
                  uint32_t wid, float* val, uint32_t* off, float* C) {
  if (!is_pow2_u32(L) || !is_pow2_u32(S) || S < 2 || S > L || scaled > 1) return ORC_ERR_ARG;
  uint64_t nc = (d + L - 1) / L;
  uint32_t per = L / S;
  const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  const float factor = scaled ? (float)S : 1.0f;
  for (uint64_t c = 0; c < nc; ++c) {
    uint64_t lo = c * L, hi = lo + L < d ? lo + L : d;
    uint32_t ctr[4] = {0xFFFFFFFFu, (uint32_t)c, wid, step};
    uint32_t rnd[4];
    orc_philox4x32_10(ctr, key, rnd);
    uint32_t o = rnd[0] % S;
    off[c] = o;
    for (uint32_t u = 0; u < per; ++u) val[c * per + u] = 0.0f;
    for (uint64_t j = lo; j < hi; ++j) {
      uint32_t t = (uint32_t)(j - lo);
      if (t % S == o) {
        float kept = factor * v[j];
        val[c * per + t / S] = kept;
        if (C) C[j] = kept;
      } else if (C) {
        C[j] = 0.0f;
      }
    }
  }
  return ORC_OK;
}

int orc_decode_rsparse(const float* val, const uint32_t* off, uint64_t d, uint32_t L, uint32_t S, float* C) {
  if (L == 0 || S == 0 || S > L) return ORC_ERR_ARG;
  uint32_t per = L / S;
  for (uint64_t j = 0; j < d; ++j) {
    uint64_t c = j / L;
    uint32_t t = (uint32_t)(j % L);
    C[j] = (t % S == off[c]) ? val[c * per + t / S] : 0.0f;
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Q = top-k sparsification (Section 3.2 "Top-k sparsification"; Section 5.1 */
/* "Top-k compression": keep the k entries largest in absolute value, zero   */
/* the rest).  Written as the definition: order all entries by (|v|          */
/* descending, index ascending) -- |v| compared through the bit pattern with */
/* the sign cleared, so +0 and -0 tie -- and keep the first k.  The payload  */
/* lists the kept entries by ascending index with their values copied        */
/* bit for bit; exactly k entries even when fewer than k are non-zero.       */
/* ------------------------------------------------------------------------ */

typedef struct { uint32_t key; uint32_t idx; } orc_keyidx;

static int cmp_key_desc_idx_asc(const void* pa, const void* pb) {
  const orc_keyidx* a = (const orc_keyidx*)pa;
  const orc_keyidx* b = (const orc_keyidx*)pb;
  if (a->key != b->key) return a->key > b->key ? -1 : 1;
  if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
  return 0;
}

int orc_q_topk(const float* v, uint64_t d, uint64_t k, uint32_t* idx, float* val, float* C) {
  if (k > d || d > 0xFFFFFFFFull) return ORC_ERR_ARG;
  orc_keyidx* order = (orc_keyidx*)malloc(sizeof(orc_keyidx) * (d ? d : 1));
  uint8_t* kept = (uint8_t*)calloc(d ? d : 1, 1);
  if (!order || !kept) { free(order); free(kept); return ORC_ERR_NOMEM; }
  for (uint64_t j = 0; j < d; ++j) {
    order[j].key = f32_bits(v[j]) & 0x7FFFFFFFu;
    order[j].idx = (uint32_t)j;
  }
  qsort(order, d, sizeof(orc_keyidx), cmp_key_desc_idx_asc);
  for (uint64_t r = 0; r < k; ++r) kept[order[r].idx] = 1;
  uint64_t m = 0;
  for (uint64_t j = 0; j < d; ++j) {
    if (kept[j]) {
      if (idx) idx[m] = (uint32_t)j;
      if (val) val[m] = v[j];
      ++m;
    }
    if (C) C[j] = kept[j] ? v[j] : 0.0f;
  }
  free(order);
  free(kept);
  return m == k ? ORC_OK : ORC_ERR_ARG;
}

int orc_decode_topk(const uint32_t* idx, const float* val, uint64_t k, uint64_t d, float* C) {
  for (uint64_t j = 0; j < d; ++j) C[j] = 0.0f;
  for (uint64_t m = 0; m < k; ++m) {
    if (idx[m] >= d) return ORC_ERR_ARG;
    C[idx[m]] = val[m];
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Q = randomised quantisation (Section 3.2 "Randomized Quantization": a     */
/* real z in [a, b] goes to a with probability (b-z)/(b-a) and to b with     */
/* probability (z-a)/(b-a); unbiased).  Reading: the low-bit grid is the     */
/* s+1 uniform magnitudes {0, q, 2q, ..., s q}, q = N/s, N the l2 norm of    */
/* the chunk of L consecutive elements the entry lies in (the normalisation  */
/* of the QSGD paper the option cites); sign kept as one bit.  With          */
/* r = |v| * (s/N), a = floor(r) and b = a+1 in grid units, so the up        */
/* probability is frac(r).  The uniform variate is a 24-bit fraction of one  */
/* Philox4x32-10 word: key = (seed low, seed high), counter = (t, chunk,     */
/* wid, step) with t = (offset in chunk)/4, the entry using output word      */
/* (offset in chunk)%4; wid = worker index, 0xFFFFFFFF on the server pass.   */
/* A chunk whose norm is zero, non-finite, or so small that s/N overflows    */
/* is sent as all zeros with a stored norm of 0.                             */
/*   lvl : d bytes, level in [0, s]                                          */
/*   sgn : ceil(d/32) words, bit = (v >= 0), layout as for sign1             */
/*   norm: ceil(d/L) floats (N, or 0 for a degenerate chunk)                 */
/* ------------------------------------------------------------------------ */

int orc_q_qsgd(const float* v, uint64_t d, uint32_t L, uint32_t s, uint64_t seed, uint32_t step,
               uint32_t wid, uint8_t* lvl, uint32_t* sgn, float* norm, float* qstep, float* C) {
  if (!is_pow2_u32(L) || L < 4 || s < 1 || s > 255) return ORC_ERR_ARG;
  uint64_t nw = (d + 31) / 32, nc = (d + L - 1) / L;
  float* sq = (float*)malloc(sizeof(float) * L);
  if (!sq) return ORC_ERR_NOMEM;
  memset(sgn, 0, sizeof(uint32_t) * nw);
  const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  const float sf = (float)s;
  const float two_m24 = 1.0f / 16777216.0f;
  for (uint64_t c = 0; c < nc; ++c) {
    uint64_t lo = c * L, hi = lo + L < d ? lo + L : d;
    uint32_t len = (uint32_t)(hi - lo);
    for (uint32_t t = 0; t < L; ++t) {
      float e = t < len ? v[lo + t] : 0.0f;
      float e2 = e * e;
      sq[t] = e2;
    }
    float ss = pairwise_sum(sq, L);
    float N = sqrtf(ss);
    float q = 0.0f, inv_q = 0.0f;
    int live = (N > 0.0f) && (N < INFINITY);
    if (live) {
      inv_q = sf / N;
      q = N / sf;
      if (!(inv_q < INFINITY)) live = 0;
    }
    if (!live) { N = 0.0f; q = 0.0f; inv_q = 0.0f; }
    norm[c] = N;
    qstep[c] = q;
    for (uint32_t t = 0; t < len; ++t) {
      uint64_t j = lo + t;
      uint32_t ctr[4] = {t / 4, (uint32_t)c, wid, step};
      uint32_t rnd[4];
      orc_philox4x32_10(ctr, key, rnd);
      uint32_t w = rnd[t % 4];
      float u = (float)(w >> 8) * two_m24; /* exact: 24-bit integer times 2^-24 */
      float a = fabsf(v[j]);
      float r = a * inv_q;
      if (r > sf) r = sf;
      float f = floorf(r);
      float p = r - f; /* exact */
      uint32_t level = (uint32_t)f + (u < p ? 1u : 0u);
      if (level > s) level = s;
      int nonneg = v[j] >= 0.0f;
      lvl[j] = (uint8_t)level;
      if (nonneg) sgn[j / 32] |= (uint32_t)1 << (j % 32);
      if (C) {
        float mag = (float)level * q;
        C[j] = nonneg ? mag : -mag;
      }
    }
  }
  free(sq);
  return ORC_OK;
}

int orc_decode_qsgd(const uint8_t* lvl, const uint32_t* sgn, const float* qstep, uint64_t d, uint32_t L,
                    float* C) {
  if (L == 0) return ORC_ERR_ARG;
  for (uint64_t j = 0; j < d; ++j) {
    float q = qstep[j / L];
    float mag = (float)lvl[j] * q;
    int nonneg = (sgn[j / 32] >> (j % 32)) & 1u;
    C[j] = nonneg ? mag : -mag;
  }
  return ORC_OK;
}


/* ------------------------------------------------------------------------ */
/* Q = ternary quantisation, the "QSGD" of Section 5.1 ("Implementations and  */
/* setups", item 2): every entry becomes -1, 0 or +1.  With m the entry of   */
/* largest absolute value of the whole vector, an entry e becomes sign(e)    */
/* with probability |e|/|m| and 0 otherwise; then one scaling factor,        */
/* magnitude of the vector over magnitude of the ternary vector, multiplies  */
/* it.  Reading: magnitudes are l1 norms (as for the 1-bit operator), so the */
/* factor is ||v||_1 / (number of non-zero entries); the sum is pairwise     */
/* over the vector padded with +0 to the next power of two.  The sign of an  */
/* entry is the bit (v >= 0).  Uniform variate: 24-bit fraction of a         */
/* Philox4x32-10 word, key = seed, counter = (j/4, 0xFFFFFFFE, wid, step),   */
/* entry j using output word j%4; the entry survives iff u < |e|/|m| (one    */
/* binary32 division), so the largest entry survives always (u < 1).  A      */
/* vector of zeros is sent as zeros with factor 0.                           */
/*   sgn : ceil(d/32) words, bit = (v >= 0)                                  */
/*   nz  : ceil(d/32) words, bit = entry is non-zero in the ternary vector   */
/*   scale: one float;  vmax: one float (|m|, for the tests that pin it)     */
/* ------------------------------------------------------------------------ */

int orc_q_ternary(const float* v, uint64_t d, uint64_t seed, uint32_t step, uint32_t wid, uint32_t* sgn,
                  uint32_t* nz, float* scale, float* vmax, float* C) {
  if (d == 0 || d > 0xFFFFFFFFull) return ORC_ERR_ARG;
  uint64_t nw = (d + 31) / 32;
  float* term = (float*)malloc(sizeof(float) * d);
  if (!term) return ORC_ERR_NOMEM;
  memset(sgn, 0, sizeof(uint32_t) * nw);
  memset(nz, 0, sizeof(uint32_t) * nw);
  const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  const float two_m24 = 1.0f / 16777216.0f;
  float m = 0.0f;
  for (uint64_t j = 0; j < d; ++j) {
    float a = fabsf(v[j]);
    term[j] = a;
    if (a > m) m = a;
  }
  float l1 = pairwise_sum_padded(term, d, next_pow2_u64(d));
  uint64_t count = 0;
  for (uint64_t j = 0; j < d; ++j) {
    uint32_t ctr[4] = {(uint32_t)(j / 4), 0xFFFFFFFEu, wid, step};
    uint32_t rnd[4];
    orc_philox4x32_10(ctr, key, rnd);
    uint32_t w = rnd[j % 4];
    float u = (float)(w >> 8) * two_m24; /* exact, in [0, 1) */
    int kept = 0;
    if (m > 0.0f) {
      float p = term[j] / m;
      kept = u < p;
    }
    if (v[j] >= 0.0f) sgn[j / 32] |= (uint32_t)1 << (j % 32);
    if (kept) {
      nz[j / 32] |= (uint32_t)1 << (j % 32);
      ++count;
    }
  }
  float s = 0.0f;
  if (count > 0) s = l1 / (float)count;
  scale[0] = s;
  if (vmax) vmax[0] = m;
  if (C) {
    for (uint64_t j = 0; j < d; ++j) {
      int kept = (nz[j / 32] >> (j % 32)) & 1u;
      int nonneg = (sgn[j / 32] >> (j % 32)) & 1u;
      C[j] = kept ? (nonneg ? s : -s) : 0.0f;
    }
  }
  free(term);
  return ORC_OK;
}

int orc_decode_ternary(const uint32_t* sgn, const uint32_t* nz, const float* scale, uint64_t d, float* C) {
  float s = scale[0];
  for (uint64_t j = 0; j < d; ++j) {
    int kept = (nz[j / 32] >> (j % 32)) & 1u;
    int nonneg = (sgn[j / 32] >> (j % 32)) & 1u;
    C[j] = kept ? (nonneg ? s : -s) : 0.0f;
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* The same passes without error compensation (Section 5.1, items 2 and 5:   */
/* "QSGD" and "Top-k SGD" compress the gradient itself and keep no error):   */
/* the vector that is compressed is g on a worker and the plain mean on the  */
/* server; no error is read, none is written.                                */
/* ------------------------------------------------------------------------ */

void orc_server_mean(const float* C_all, uint32_t n, uint64_t d, float* v) {
  float one = 1.0f;
  float inv_n = one / (float)n;
  for (uint64_t j = 0; j < d; ++j) {
    float acc = 0.0f;
    for (uint32_t i = 0; i < n; ++i) {
      float t = acc + C_all[(uint64_t)i * d + j];
      acc = t;
    }
    float mean = acc * inv_n;
    v[j] = mean;
  }
}
