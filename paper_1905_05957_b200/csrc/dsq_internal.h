// Host-side launch interface shared by the kernel translation units and the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/dsq.h"
#include "dsq_common.cuh"

namespace dsq {

// Kernels launched by this library since it was loaded (reported by ds_kernel_launches()).
extern std::atomic<uint64_t> g_kernel_launches;
inline void count_launches(uint64_t n) { g_kernel_launches.fetch_add(n, std::memory_order_relaxed); }

// Records the text of a CUDA error for ds_last_error() (kept per host thread) and returns DS_ERR_CUDA.
int cuda_fail(cudaError_t e, const char* where);

// Runs X(S) for the source kind `srck` with S a compile-time constant; returns
// cudaErrorInvalidValue from the enclosing function for an unknown kind.
#define DSQ_SWITCH_SRC(srck, X)                          \
  switch (srck) {                                        \
    case SRC_WORKER: X(SRC_WORKER); break;               \
    case SRC_SRV_IDENTITY: X(SRC_SRV_IDENTITY); break;   \
    case SRC_SRV_SIGN1: X(SRC_SRV_SIGN1); break;         \
    case SRC_SRV_TOPK: X(SRC_SRV_TOPK); break;           \
    case SRC_SRV_QSGD: X(SRC_SRV_QSGD); break;           \
    case SRC_SRV_CLIP: X(SRC_SRV_CLIP); break;           \
    case SRC_SRV_RSPARSE: X(SRC_SRV_RSPARSE); break;     \
    case SRC_WORKER_PLAIN: X(SRC_WORKER_PLAIN); break;   \
    case SRC_SRV_TERNARY: X(SRC_SRV_TERNARY); break;     \
    default: return cudaErrorInvalidValue;               \
  }

// kernel<<<grid, block, 0, st>>>(args...) with programmatic stream serialization allowed (the
// kernel begins with pdl_prologue()).  A failed launch shows in cudaGetLastError().
template <typename... P, typename... A>
inline void launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, cudaStream_t st, A&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// The same with `smem` bytes of dynamic shared memory (beyond the 48 KB a kernel gets by default the
// limit is raised first; that call only sets a number on the host).
template <typename... P, typename... A>
inline void launch_pdl_smem(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
  if (smem > 48 * 1024) (void)cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// Destination of a chunk-wise operator (SIGN1 or QSGD).
struct ChunkParams {
  uint32_t* out_bits;        // sign words, row stride bits_stride (in words)
  float* out_scale;          // SIGN1: scale per chunk; QSGD: grid step q per chunk; row stride scale_stride (floats)
  uint8_t* out_lvl;          // QSGD: level bytes, row stride lvl_stride (bytes)
  uint64_t bits_stride, scale_stride, lvl_stride;
  float* delta_out;          // residual destination, row stride delta_row_stride (floats)
  uint64_t delta_row_stride;
  float* x;                  // non-NULL: fused model update (server pass)
  float gamma;
  float levels_f;            // QSGD: s
  uint32_t levels_u;
  PhiloxKeys keys;           // Philox round keys
  uint32_t step;             // the step word of the counter
  uint32_t server_pass;      // 1: counter word 2 is 0xFFFFFFFF, else the row (worker) index
  uint32_t log2G;            // filled by the launcher
  uint32_t chunk0;           // index of the pass's first chunk in the whole vector (a pass over a slice of d)
  uint32_t row0;             // worker index of the pass's first row (a pass over some of the workers)
  uint32_t sign_l2;          // SIGN1: 1 = the scale is ||v_c||_2 / sqrt(len_c) instead of ||v_c||_1 / len_c
};

// Destination of a decoded payload for the dense model update.
struct PayloadView {
  int op;
  const uint8_t* base;
  uint64_t off[3];
  uint32_t log2_chunk;
  float levels_f;
  uint32_t clip_bits;
  uint32_t log2_keep;
  uint64_t k;
};

// Per-vector state of the radix select (device memory inside the workspace).
struct TopkState {
  uint32_t k_rem;      // entries still to take inside the current threshold bin
  uint32_t tb1, tb2;   // threshold digits: key bits 30..19 and 18..7
  uint32_t tau;        // full 31-bit key of the k-th largest entry
  uint32_t r;          // how many entries with key == tau are kept (lowest indices first)
  uint32_t total_gt, total_tie;
  uint32_t reserved0;
  uint32_t need_full;  // 1: the candidates pass1 listed (if any) did not contain the k-th entry
  uint32_t zeroed_above;  // entries with a key above this were zeroed in the residual when they were listed
};

// Threshold history of one vector (the keys tau of the two previous steps), kept across steps so
// that pass1 can mark candidates itself.
struct TopkPred {
  uint32_t magic, tau_last, tau_prev, err;
};

// Carving of the workspace for `rows` simultaneous selections over d-vectors.
struct TopkPlan {
  uint64_t d, k;
  uint32_t rows;
  uint64_t nseg;        // 32768-entry segments per vector
  uint64_t bm_stride;   // bitmap words per vector (whole segments)
  uint64_t ntile;       // 4096-entry tiles per vector
  uint64_t list_cap;    // slots of the candidate list per vector (0: no list, gather instead)
  uint64_t off_hist, off_list_count, off_state, off_bm_gt, off_bm_eq, off_seg, off_list, off_tile_info, off_dense;
  uint64_t bytes;
  TopkPred* pred;       // [rows] history outside the scratch (device memory), or NULL: no prediction
};

struct TopkIO {
  uint32_t* idx;            // payload sub-arrays of row 0; rows are payload_stride bytes apart
  float* val;
  uint64_t payload_stride;
  float* v_inout;           // [rows, d]: receives v, then has the kept entries zeroed (the residual).  With
                            // keep_error = 0 (source SRC_WORKER_PLAIN): where v already lies (the gradient); only read
  int keep_error;
  uint32_t* span_off;       // non-NULL: also receives, per vector, where every span of kSparseSpan indices begins in
                            // the emitted index list ([rows, nspan + 1]; the table launch_sparse_accumulate works from)
  float* x;                 // non-NULL: fused model update at the kept entries (server pass)
  float gamma;
  uint32_t* dev_status;
};

void topk_plan(uint64_t d, uint32_t rows, uint64_t k, bool with_list, TopkPlan* plan);
cudaError_t launch_topk(int src_kind, const SrcParams& src, const TopkPlan& plan, void* workspace, const TopkIO& io,
                        uint32_t rows, uint64_t k, cudaStream_t st);

// The selection over ONE slice of a vector that lives on several GPUs, stage by stage (see
// ds_server_topk_slice_* in dsq.h): the scratch is carved from the start of `workspace`.
uint64_t topk_slice_workspace_bytes(uint64_t d_slice, uint64_t k);
cudaError_t launch_topk_slice_begin(int src_kind, const SrcParams& src, void* workspace, float* v_out, uint64_t k,
                                    uint32_t* hist_out, cudaStream_t st);
cudaError_t launch_topk_slice_digit(int level, void* workspace, const float* v, uint64_t d_slice, int vec, uint64_t k,
                                    uint32_t* hist_sum, uint32_t* hist_next, cudaStream_t st);
cudaError_t launch_topk_slice_emit(void* workspace, float* v_io, uint64_t d_slice, uint64_t k, uint32_t ties_to_keep,
                                   uint32_t count, uint32_t idx_base, uint32_t* out_idx, float* out_val, float* x, float gamma,
                                   cudaStream_t st);

cudaError_t launch_chunked(int op, int src_kind, const SrcParams& src, const ChunkParams& p, uint32_t rows,
                           uint32_t chunk, cudaStream_t st);

// Q = identity: payload c = v, residual +0, optional fused update.
cudaError_t launch_identity(int src_kind, const SrcParams& src, float* out_c, uint64_t c_row_stride, float* delta_out,
                            uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st);

// Q = clipping: payload hi = bits(v) >> bits (16- or 8-bit entries), residual v - Q[v], optional fused update.
cudaError_t launch_clip(int src_kind, const SrcParams& src, uint32_t bits, uint8_t* out_hi, uint64_t hi_row_stride,
                        float* delta_out, uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st);

// Q = randomised sparsification: one entry in 2^log2_keep of every chunk survives (see include/dsq.h).
struct RsparseParams {
  float* out_val;            // survivors, row stride val_stride (floats)
  uint32_t* out_off;         // the draw of every chunk, row stride off_stride (words)
  uint64_t val_stride, off_stride;
  uint32_t log2_chunk, log2_keep, scaled;
  PhiloxKeys keys;
  uint32_t step, server_pass;
  uint32_t chunk0, row0;     // a pass over a slice of d / some of the workers: index of its first chunk / worker
};
cudaError_t launch_rsparse(int src_kind, const SrcParams& src, const RsparseParams& rp, float* delta_out,
                           uint64_t delta_row_stride, float* x, float gamma, uint32_t rows, cudaStream_t st);

// Operators with ONE factor for the whole vector: the 1-bit operator as Section 3.2 / Section 5.1 state
// it (chunk = 0) and the ternary quantiser of Section 5.1, item 2.  The factor depends on a sum (and,
// ternary, on the largest magnitude and the number of survivors) over all d entries, so a pass is
// several kernels: tile sums, their pairwise combination, then the encoding.  v is recomputed from its
// source in every kernel instead of being stored.
struct WholeParams {
  uint32_t* out_sgn;         // sign words (bit = v >= 0), row stride word_stride (in words)
  uint32_t* out_nz;          // ternary: words of the non-zero plane
  float* out_scale;          // one factor per row, row stride word_stride (floats)
  uint64_t word_stride;
  float* delta_out;          // residual destination, or NULL: no error is kept
  uint64_t delta_row_stride;
  float* x;                  // non-NULL: fused model update (server pass)
  float gamma;
  PhiloxKeys keys;
  uint32_t step, server_pass;
  uint32_t l2;               // SIGN1: 1 = l2 magnitudes
};
uint64_t whole_workspace_bytes(uint64_t d, uint32_t rows);
cudaError_t launch_whole(int op, int src_kind, const SrcParams& src, const WholeParams& p, void* workspace, uint32_t rows,
                         cudaStream_t st);

// x = x - gamma * decode(payload)
cudaError_t launch_apply(const PayloadView& pv, float* x, uint64_t d, float gamma, cudaStream_t st);

// acc[j] = sum over workers i = 0..n-1, in that order, of the value worker i's sparse payload holds for j
// (every entry of acc is written).  offsets: scratch of sparse_offsets_bytes(n, d) bytes; offsets_ready: the
// table in it is already filled (by the top-k pass that wrote these payloads), else it is built first.
constexpr uint32_t kSparseSpan = 8192;   // indices per span of the table
uint64_t sparse_offsets_bytes(uint32_t n, uint64_t d);
cudaError_t launch_sparse_accumulate(const uint8_t* wp, uint64_t stride, uint64_t off_idx, uint64_t off_val, uint32_t n,
                                     uint64_t k, uint64_t d, uint32_t* offsets, bool offsets_ready, float* acc, cudaStream_t st);

}  // namespace dsq
