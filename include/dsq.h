/*
 * dsq.h -- C ABI of the DoubleSqueeze step library (CUDA, sm_100a).
 *
 * One iteration of DoubleSqueeze (Algorithm 1 of arXiv:1905.05957) with the n
 * workers held as the rows of one [n, d] fp32 tensor on a single GPU:
 *
 *   worker  i :  v_i = g_i + delta_i          (Section 3.1, Eq. 2)
 *                send Q[v_i]                  (Algorithm 1, "Compress")
 *                delta_i = v_i - Q[v_i]       (Eq. 3)
 *   server    :  v = delta + (1/n) sum_i Q[v_i]
 *                send Q[v];  delta = v - Q[v] (Eq. 4)
 *   worker    :  x = x - gamma Q[v]           (Algorithm 1, "Update the local model")
 *
 * Q is one of the compression options of Section 3.2 / Section 5.1; the worker
 * pass and the server pass may use different ones.
 *
 * General rules
 *  - Every pointer in ds_buffers, and the gradient g, is DEVICE memory owned by
 *    the caller.  The library allocates no device memory and keeps no copy of g.
 *    The handle is host memory only.
 *  - ds_worker_compress / ds_server_aggregate_compress / ds_apply_update only
 *    enqueue work on the given CUDA stream (a cudaStream_t passed as void*; NULL
 *    is the default stream); they never synchronise.  One handle must be used on
 *    one stream at a time.
 *  - Every function returns a ds_status.  Nothing throws across the boundary.
 *    Conditions detected on the device are OR-ed into dev_status[0] (DS_DEV_*),
 *    which the caller reads when it chooses; kernels never trap.
 *  - All multi-byte payload fields are little-endian; all arithmetic is IEEE-754
 *    binary32 round-to-nearest-even with no fused multiply-add.
 */
#ifndef DSQ_H_
#define DSQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ds_ctx* ds_handle;

typedef enum {
  DS_OK = 0,
  DS_NEED_BUFFERS = 1,          /* ds_create in query mode: *_bytes filled, no handle made */
  DS_ERR_INVALID_ARG = -1,
  DS_ERR_ALIGN = -2,            /* a buffer is not 16-byte aligned */
  DS_ERR_BUFFER_TOO_SMALL = -3,
  DS_ERR_STATE = -4,            /* calls out of order within a step */
  DS_ERR_CUDA = -5,             /* a launch failed; see ds_last_error() */
  DS_ERR_UNSUPPORTED = -6
} ds_status;

/* dev_status is four words.  Word 0 holds flags: */
#define DS_DEV_TOPK_INCONSISTENT 0x1u /* top-k selection counted a number of entries other than k */
/* Words 1 and 2 count top-k selections (one per vector and pass) by the route they took: with the
 * threshold band predicted from the previous steps ("predicted": v is read once), or through the
 * full histogram after a missing or wrong prediction ("full": v is read three times).  Both routes
 * give the same result; the counters are for tests and tuning.  Word 3 is reserved. */
#define DS_DEV_WORD_FLAGS 0
#define DS_DEV_WORD_TOPK_PREDICTED 1
#define DS_DEV_WORD_TOPK_FULL 2

/* flags of ds_server_aggregate_compress */
#define DS_FUSE_APPLY 0x1u /* also perform x = x - gamma Q[v]; ds_apply_update is then not called */

/*
 * Compression operators.
 *
 * DS_Q_IDENTITY  Q[v] = v.  The step is then plain parallel SGD (Section 1).
 *
 * DS_Q_SIGN1     "1-bit compression" of Section 5.1 (Section 3.2 "1-Bit Quantization"): the sign
 *                of every entry plus a scaling factor that restores the magnitude.  Here the
 *                factor is the mean absolute value of each chunk of `chunk` consecutive entries
 *                of the flat vector (the last chunk may be short; its true length divides).
 *                bit = (v >= 0);  Q[v]_j = bit ? +s_c : -s_c.
 *                With norm = DS_NORM_L2 the magnitudes of Section 5.1's ratio are l2 norms (the
 *                norm Section 3.2 prints): s_c = ||v_c||_2 / sqrt(len_c).  Same payload format.
 *
 * DS_Q_TOPK      "Top-k compression" of Section 5.1 (Section 3.2 "Top-k sparsification"): the k
 *                entries of largest absolute value over the whole d-vector keep their value, all
 *                others become 0.  Equal magnitudes are taken by lower index first.  Always
 *                exactly k entries.
 *
 * DS_Q_QSGD      "Randomized Quantization" of Section 3.2: |v_j| is rounded at random to one of
 *                its two neighbours on the grid {0, q, ..., levels*q}, q = N_c / levels, with the
 *                probabilities that make it unbiased; N_c is the l2 norm of the entry's chunk of
 *                `chunk` consecutive entries; the sign is kept.  Randomness: Philox4x32-10,
 *                key = (seed low, seed high), counter = (offset_in_chunk/4, chunk index, worker
 *                index or 0xFFFFFFFF on the server pass, step); entry uses output word
 *                offset_in_chunk%4, top 24 bits, as a uniform in [0,1).
 *
 * DS_Q_CLIP      "Clipping" of Section 3.2: the low `levels` bits (16 or 24) of every binary32 number
 *                are set to zero, which keeps the sign, the exponent and the leading fraction
 *                bits (truncation toward zero); deterministic and biased.  The payload carries
 *                the surviving high 32 - levels bits of every entry.  The residual v - Q[v] is
 *                exact.
 *
 * DS_Q_RSPARSE   "Randomized Sparsification" of Section 3.2: a number survives with probability 1/S
 *                (S = `levels`, a power of two) and becomes 0 otherwise.  The entries of a chunk of
 *                `chunk` consecutive entries share one draw o, uniform in 0..S-1 (Philox4x32-10,
 *                key = seed, counter = (0xFFFFFFFF, chunk index, worker index or 0xFFFFFFFF on
 *                the server pass, step), first output word mod S): the entry at offset t of its
 *                chunk survives iff t mod S == o, so each entry survives with probability exactly
 *                1/S and a chunk always sends chunk/S values.  norm = DS_RSPARSE_SCALED: survivors
 *                are multiplied by S, the unbiased form the paper prints (no contraction: its
 *                compensated error grows; offered for completeness).  norm = DS_RSPARSE_PLAIN:
 *                survivors keep their value (a contraction).
 *
 * DS_Q_SIGN1 with chunk = 0: the 1-bit operator exactly as Section 3.2 and Section 5.1 state it, with ONE
 *                factor for the whole vector: ||v||_1 / d, or ||v||_2 / sqrt(d) with norm = DS_NORM_L2.  The
 *                factor needs a sum over all of v first, so a pass is three kernels and reads its inputs
 *                twice (about 20 bytes per entry on a worker instead of 12).
 *
 * DS_Q_TERNARY   the "QSGD" of Section 5.1 ("Implementations and setups", item 2): with m the entry of
 *                largest absolute value of the whole vector, an entry e becomes sign(e) with probability
 *                |e| / |m| and 0 otherwise; one factor, the l1 magnitude of v over that of the ternary
 *                vector (||v||_1 / number of non-zeros), multiplies it.  The sign of an entry is the bit
 *                (v >= 0).  Randomness: Philox4x32-10, key = seed, counter = (j/4, 0xFFFFFFFE, worker
 *                index or 0xFFFFFFFF on the server pass, step); entry j uses output word j%4, top 24 bits,
 *                as a uniform u in [0,1), and survives iff u < |e| / |m| (so the largest entry always
 *                does).  chunk must be 0.  Five kernels per pass, inputs read three times.
 *
 * Chunk reductions (sum of |v| or of v*v) are pairwise sums in index order over the chunk padded
 * with zeros to `chunk` entries (whole vector: to the next power of two at or above d), so results do not
 * depend on launch geometry.
 */
typedef enum {
  DS_Q_IDENTITY = 0, DS_Q_SIGN1 = 1, DS_Q_TOPK = 2, DS_Q_QSGD = 3, DS_Q_CLIP = 4, DS_Q_RSPARSE = 5, DS_Q_TERNARY = 6
} ds_op;

/* ds_qspec.norm for DS_Q_SIGN1 */
#define DS_NORM_L1 0u /* s_c = ||v_c||_1 / len_c (also selected by 1) */
#define DS_NORM_L2 2u /* s_c = ||v_c||_2 / sqrt(len_c) */
/* ds_qspec.norm for DS_Q_RSPARSE */
#define DS_RSPARSE_PLAIN 0u  /* survivors keep their value */
#define DS_RSPARSE_SCALED 1u /* survivors are multiplied by S */

typedef struct {
  int32_t op;        /* ds_op */
  uint32_t chunk;    /* SIGN1, QSGD, RSPARSE: a power of two in [128, 8192]; SIGN1 also 0 = one factor for the
                        whole vector; TERNARY: 0; else ignored */
  uint64_t k;        /* TOPK: 0 <= k <= d; else ignored */
  uint32_t levels;   /* QSGD: 1 <= levels <= 255; CLIP: bits set to zero, 16 or 24;
                        RSPARSE: S, a power of two in [2, 128]; else ignored */
  uint32_t norm;     /* SIGN1: DS_NORM_L1 (0 or 1) or DS_NORM_L2 (2); RSPARSE: DS_RSPARSE_*; else must be 0 */
} ds_qspec;

/*
 * ds_config.flags.  DS_NO_COMPENSATION: the methods of Section 5.1 that compress without keeping the error
 * ("Top-k SGD", item 5; "QSGD", item 2, with DS_Q_TERNARY workers and an IDENTITY server): a worker sends
 * Q[g_i], the server sends Q[(1/n) sum_i Q[g_i]], x = x - gamma * that.  No error is read and none is
 * written: delta_w is not used at all (delta_w_bytes is 0, the pointer may be NULL) and the worker pass
 * moves 4 bytes per entry plus the payload instead of 12.  delta_s is likewise unused, except that a TOPK
 * server pass lays its vector out there (delta_s then is scratch: required, never read back by a later
 * step); for every other server operator delta_s_bytes is 0.
 */
#define DS_NO_COMPENSATION 0x1u

typedef struct {
  uint32_t n;        /* workers, 1 <= n <= 65535 */
  uint32_t delta_w_rows; /* 0 (or n): delta_w holds the errors of all n workers.  R < n: this instance is one rank of
                        a deployment with one or a few workers per GPU and keeps the errors of R consecutive workers
                        only (delta_w is float[R*d]; worker i uses row i mod R, and a ds_worker_compress_rows call
                        must stay inside one block of R workers that starts at a multiple of R); ds_worker_compress
                        for all n workers is then DS_ERR_UNSUPPORTED.  The payload buffers keep their n rows */
  uint64_t d;        /* model dimension, 1 <= d < 2^32 */
  float gamma;       /* learning rate, finite */
  uint32_t flags;    /* DS_NO_COMPENSATION or 0 */
  ds_qspec worker_q; /* Q of the worker pass */
  ds_qspec server_q; /* Q of the server pass */
  uint64_t seed;     /* Philox key for DS_Q_QSGD */
} ds_config;

/*
 * Caller-owned device buffers.  Layouts:
 *   x        float[d]        model; the caller sets x_0
 *   delta_w  float[n*d]      worker errors, row i = worker i (float[R*d] with delta_w_rows = R); the caller zero-fills (delta = 0)
 *   delta_s  float[d]        server error; the caller zero-fills
 *   worker_payload           n payloads at a fixed stride, see ds_get_layout()
 *   server_payload           one payload
 *   workspace                scratch of the top-k path and of the whole-vector operators; may be NULL when
 *                            workspace_bytes is 0.
 *                            Zero-fill it once.  Between calls it holds only hints (the previous
 *                            steps' threshold bins); whatever it holds, results are the same
 *   dev_status uint32[4]     the caller zero-fills (flags and counters, see DS_DEV_*)
 * Every non-NULL pointer must be 16-byte aligned and at least *_bytes long (dev_status: 4-byte aligned).
 */
typedef struct {
  float* x;
  float* delta_w;
  float* delta_s;
  void* worker_payload;
  void* server_payload;
  void* workspace;
  uint32_t* dev_status;
  size_t x_bytes, delta_w_bytes, delta_s_bytes;
  size_t worker_payload_bytes, server_payload_bytes, workspace_bytes;
} ds_buffers;

/*
 * Byte layout of one payload.  `stride` is the distance between consecutive workers' payloads
 * (for the server payload: its total size).  Sub-array i starts `off[i]` bytes into the payload,
 * is 16-byte aligned and holds `count[i]` elements:
 *   IDENTITY  [0] float c[d]
 *   SIGN1     [0] uint32 bits[ceil(d/32)]  entry j -> bit j%32 of word j/32, pad bits 0
 *             [1] float  scale[ceil(d/chunk)]
 *   TOPK      [0] uint32 idx[k] ascending  [1] float val[k] (bit copies of v[idx])
 *   QSGD      [0] uint8  lvl[d]            [1] uint32 sgn[ceil(d/32)] (bit = v >= 0)
 *             [2] float  step[ceil(d/chunk)] (the grid step q = N_c / levels that multiplies the
 *                 levels; 0 for a chunk sent as all zeros)
 *   CLIP      [0] uint16 hi[d] (levels = 16) or uint8 hi[d] (levels = 24): bits(v) >> levels
 *   SIGN1, chunk = 0: as SIGN1 with one float in scale
 *   TERNARY   [0] uint32 sgn[ceil(d/32)] (bit = v >= 0)  [1] uint32 nz[ceil(d/32)] (bit = entry is non-zero)
 *             [2] float  scale[1]
 *   RSPARSE   [0] float  val[ceil(d/chunk) * chunk/S]  slot j/S = Q[v]_j of the survivor j, +0 where j >= d
 *             [1] uint32 off[ceil(d/chunk)]            the draw o of every chunk
 */
typedef struct {
  uint64_t stride;
  uint64_t off[3];
  uint64_t count[3];
} ds_payload_layout;

/* Host-only.  which = 0: worker payload, 1: server payload.  DS_ERR_INVALID_ARG on a bad config. */
int ds_get_layout(const ds_config* cfg, int which, ds_payload_layout* out);

/*
 * Algorithm 1, "Input": fixes n, d, gamma and the operators.  Host-only; launches nothing.
 * Query mode: with bufs->x == NULL every *_bytes field of *bufs is filled and DS_NEED_BUFFERS is
 * returned (handle untouched).  Otherwise pointers and sizes are checked (DS_ERR_INVALID_ARG,
 * DS_ERR_ALIGN, DS_ERR_BUFFER_TOO_SMALL) and a handle is returned in *out.
 */
int ds_create(const ds_config* cfg, ds_buffers* bufs, ds_handle* out);

/*
 * Algorithm 1, "On worker" (Eq. 2, compress, Eq. 3) for all n workers.
 * g: device float[n*d], row i = gradient of worker i; read once, not retained.
 * step: iteration number t (enters the random stream only).
 * Writes worker_payload and delta_w.  DS_ERR_STATE unless the previous step is complete.
 */
int ds_worker_compress(ds_handle h, const float* g, uint32_t step, void* cuda_stream);

/*
 * Algorithm 1, "On parameter server" (Eq. 4): decode the n worker payloads, average in worker
 * order, add delta_s, compress, keep the residual.  Writes server_payload and delta_s; with
 * DS_FUSE_APPLY also updates x and completes the step.  DS_ERR_STATE unless ds_worker_compress
 * was the previous call.  worker_payload and workspace are read as that call left them (a TOPK worker pass
 * leaves an index of its payloads in the workspace): do not modify either between the two calls.
 */
int ds_server_aggregate_compress(ds_handle h, uint32_t step, uint32_t flags, void* cuda_stream);

/*
 * Algorithm 1, "Update the local model": x = x - gamma Q[v], decoded from server_payload.
 * DS_ERR_STATE unless an unfused ds_server_aggregate_compress was the previous call.
 */
int ds_apply_update(ds_handle h, void* cuda_stream);

/* Frees the host handle.  Device buffers stay the caller's. */
int ds_destroy(ds_handle h);

/*
 * The same two passes for a deployment in which every GPU is one worker and owns one slice of the
 * server (Section 3.1 notes that the method is not tied to a single parameter server): each
 * rank runs the worker pass for its own rows, receives the other workers' payload slices into its
 * worker_payload buffer, runs the server pass over its slice of d, and applies the update from the
 * server payload slices it gathered.  Moving the slices between GPUs is the caller's business.
 *
 * ds_worker_compress_rows: Algorithm 1, "On worker", for workers row0 .. row0+nrows-1 only; g holds
 *   those nrows rows ([nrows, d] device memory).  delta_w and worker_payload keep their [n, ...]
 *   layout; only the named rows are read and written.  Randomised operators draw with the global
 *   worker index, so the result equals what ds_worker_compress gives for these rows.
 * ds_server_aggregate_compress_slice: Algorithm 1, "On parameter server" (Eq. 4), for the entries
 *   lo .. hi-1 of every vector: decodes that slice of all n worker payloads, writes that slice of
 *   delta_s and of the server payload and, with DS_FUSE_APPLY, of x.  lo must be a multiple of
 *   DS_SLICE_ALIGN, hi a multiple of it or d.  The union of disjoint slices covering [0, d) equals
 *   one ds_server_aggregate_compress bit for bit.
 * ds_apply_update_slice: x = x - gamma Q[v] on lo .. hi-1 from that slice of the server payload.
 *
 * Operators that act per chunk or per entry (IDENTITY, SIGN1 with a chunk, QSGD, CLIP, RSPARSE) are supported on
 * both passes; the operators that need a quantity of the whole vector (TOPK, SIGN1 with chunk = 0, TERNARY) on
 * either pass are DS_ERR_UNSUPPORTED here (a TOPK server pass over slices has calls of its own, below).  These calls do not take part in the worker -> server -> apply order check
 * of the whole-vector calls: the caller sequences its slices.  Errors as for the whole-vector calls.
 */
#define DS_SLICE_ALIGN 8192u
int ds_worker_compress_rows(ds_handle h, const float* g, uint32_t row0, uint32_t nrows, uint32_t step, void* cuda_stream);
int ds_server_aggregate_compress_slice(ds_handle h, uint32_t step, uint32_t flags, uint64_t lo, uint64_t hi,
                                       void* cuda_stream);
int ds_apply_update_slice(ds_handle h, uint64_t lo, uint64_t hi, void* cuda_stream);

/*
 * Top-k on the server pass (Section 3.2, "Top-k sparsification": the k largest entries of the WHOLE vector) when the
 * server's vector is spread over several GPUs, slice lo .. hi-1 on this one.  The threshold is a property of the whole
 * vector, so the selection is cut into stages at the points where a histogram over all slices is needed; between the
 * stages the caller adds the slices' histograms up across the GPUs (an all-reduce of 4096 words) and hands the sum to
 * every slice.  Worker payloads must be of an operator that is laid out along d (everything but TOPK and the
 * whole-vector operators).  The result equals ds_server_aggregate_compress on the whole vector bit for bit.
 *
 *  1. ds_server_topk_slice_begin   v = delta_s + (1/n) sum_i Q[v_i] on the slice (Eq. 4), written over that slice of
 *                                  delta_s; hist[b] = how many of the slice's entries have (bits(v) & 0x7fffffff) >> 19 == b.
 *  2. ds_server_topk_slice_digit   level 1, 2, 3: hist_sum = the sum over all slices of the previous stage's histogram
 *                                  (the call consumes and clears it).  Picks this digit of the threshold (12, 12 and 7
 *                                  key bits) and writes the next stage's histogram of this slice into hist_next.  After
 *                                  level 3, hist_next[0..3] = (entries of this slice above the threshold tau, entries
 *                                  equal to it, the number r of entries equal to tau that the whole vector keeps, tau).
 *  3. ds_server_topk_slice_emit    ties go to lower indices first, so the caller gives slice q the quota
 *                                  ties_to_keep = clamp(r - ties in the slices before q, 0, ties in q); the slice then
 *                                  keeps count = above + ties_to_keep entries.  Writes them (GLOBAL indices ascending,
 *                                  values) into slots first_slot .. first_slot+count-1 of the server payload's idx / val
 *                                  arrays (first_slot = the counts of the slices before q, so the gathered payload is
 *                                  the whole vector's), zeroes them in delta_s, and with DS_FUSE_APPLY updates x there.
 *  4. ds_apply_update_sparse_range x = x - gamma Q[v] for the entries in slots first_slot .. +count-1 of the server
 *                                  payload (the parts gathered from the other slices).
 * hist, hist_sum, hist_next: device uint32[4096], 16-byte aligned, the caller's.  The stages keep their state in the
 * workspace; one slice at a time per handle.  Errors as for the slice calls above.
 */
int ds_server_topk_slice_begin(ds_handle h, uint32_t step, uint64_t lo, uint64_t hi, uint32_t* hist, void* cuda_stream);
int ds_server_topk_slice_digit(ds_handle h, int level, uint64_t lo, uint64_t hi, uint32_t* hist_sum, uint32_t* hist_next,
                               void* cuda_stream);
int ds_server_topk_slice_emit(ds_handle h, uint64_t lo, uint64_t hi, uint32_t ties_to_keep, uint32_t count, uint64_t first_slot,
                              uint32_t flags, void* cuda_stream);
int ds_apply_update_sparse_range(ds_handle h, uint64_t first_slot, uint64_t count, void* cuda_stream);

/*
 * Convenience for callers that hold data in HOST memory: copies g_host (float[n*d], ideally
 * pinned) into the caller's device staging buffer g_dev, runs worker + server(+fused apply), and
 * copies the server payload and/or x back to host if the respective pointer is non-NULL.  All
 * on `cuda_stream`, asynchronously; the caller synchronises the stream before reading.
 */
int ds_step_host(ds_handle h, const float* g_host, float* g_dev, uint32_t step, void* server_payload_host,
                 float* x_host, void* cuda_stream);

/*
 * (No counterpart in the paper: a packaging variant of the top-k worker step for one vector.)
 *
 * For callers that must not allocate device memory where they compress -- inside a stream
 * capture, as a plug-in of a framework that owns the memory pool, or in a loop where allocation is
 * forbidden after start-up -- and therefore cannot provide the top-k workspace that ds_create asks
 * for.  Computes, for ONE vector,  v = g + delta,  (idx, val) = top-k of v (same rules as
 * DS_Q_TOPK),  delta = v - Q[v],  using scratch memory that is a fixed array inside the library.
 *
 *   g, delta   device float[d]; delta is read and overwritten in place
 *   idx, val   device uint32[k], float[k]: ascending indices and the values kept
 *   dev_status device uint32[1], zero-filled by the caller; DS_DEV_* bits are OR-ed in
 *
 * Limits and rules:
 *  - d <= DS_STATIC_TOPK_MAX_D, else DS_ERR_UNSUPPORTED and nothing is launched.  The array costs
 *    about 2 MiB of device memory on every GPU that loads the library, until the process exits.
 *  - Calls no cudaMalloc/cudaFree and no allocating library routine.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls share the one array: two calls whose kernels may overlap on the GPU (different
 *    streams, no dependency between them) race.  Issue them on one stream or order them.
 *  - Asynchronous on cuda_stream like the other calls; pointers must be 4-byte aligned (16-byte
 *    aligned g and delta with d % 4 == 0 take the vector path).
 */
#define DS_STATIC_TOPK_MAX_D (1u << 23)
int ds_topk_worker_static(const float* g, float* delta, uint64_t d, uint64_t k, uint32_t* idx, float* val,
                          uint32_t* dev_status, void* cuda_stream);

/* Text of the most recent CUDA error seen by this thread's calls ("" if none). */
const char* ds_last_error(void);

/* Number of kernels this library has launched since it was loaded (all handles, all streams). */
uint64_t ds_kernel_launches(void);

/* Library version, major*100 + minor. */
int ds_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DSQ_H_ */
