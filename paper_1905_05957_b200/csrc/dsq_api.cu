// C ABI of the DoubleSqueeze step library: argument checking, payload layout, and the dispatch of
// each call of Algorithm 1 onto the kernels.  Host code only; no device memory is allocated here.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "dsq_internal.h"

using namespace dsq;

namespace {
thread_local char g_last_error[256] = "";
}

namespace dsq {
std::atomic<uint64_t> g_kernel_launches{0};

int cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_last_error, sizeof g_last_error, "%s: %s", where, cudaGetErrorString(e));
  return DS_ERR_CUDA;
}
}  // namespace dsq

namespace {

inline uint64_t round16(uint64_t b) { return (b + 15u) & ~uint64_t(15); }
inline bool is_pow2(uint32_t x) { return x && !(x & (x - 1)); }
inline uint32_t log2u(uint32_t x) { uint32_t l = 0; while ((1u << l) < x) ++l; return l; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool qspec_ok(const ds_qspec& q, uint64_t d) {
  if (q.op == DS_Q_SIGN1 ? (q.norm != DS_NORM_L1 && q.norm != 1u && q.norm != DS_NORM_L2)
                         : (q.op == DS_Q_RSPARSE ? q.norm > DS_RSPARSE_SCALED : q.norm != 0))
    return false;
  switch (q.op) {
    case DS_Q_IDENTITY: return true;
    case DS_Q_SIGN1: return q.chunk == 0 || (is_pow2(q.chunk) && q.chunk >= 128 && q.chunk <= 8192);
    case DS_Q_TERNARY: return q.chunk == 0;
    case DS_Q_QSGD: return is_pow2(q.chunk) && q.chunk >= 128 && q.chunk <= 8192 && q.levels >= 1 && q.levels <= 255;
    case DS_Q_TOPK: return q.k <= d;
    case DS_Q_CLIP: return q.levels == 16 || q.levels == 24;
    case DS_Q_RSPARSE:
      return is_pow2(q.chunk) && q.chunk >= 128 && q.chunk <= 8192 && is_pow2(q.levels) && q.levels >= 2 && q.levels <= 128;
    default: return false;
  }
}

bool config_ok(const ds_config* c) {
  if (!c) return false;
  if (c->n < 1 || c->n > 65535 || c->delta_w_rows > c->n || (c->flags & ~DS_NO_COMPENSATION)) return false;
  if (c->d < 1 || c->d >= (1ull << 32)) return false;
  if (!std::isfinite(c->gamma)) return false;
  return qspec_ok(c->worker_q, c->d) && qspec_ok(c->server_q, c->d);
}

// Operators whose scaling factor belongs to the whole vector (several kernels per pass, not sliceable).
bool whole_vector(const ds_qspec& q) { return (q.op == DS_Q_SIGN1 && q.chunk == 0) || q.op == DS_Q_TERNARY; }

bool no_compensation(const ds_config& c) { return (c.flags & DS_NO_COMPENSATION) != 0; }

// Rows of delta_w this instance holds: all n, or the R workers of its own block.
uint32_t delta_rows(const ds_config& c) { return c.delta_w_rows ? c.delta_w_rows : c.n; }

void layout_of(const ds_qspec& q, uint64_t d, ds_payload_layout* L) {
  memset(L, 0, sizeof *L);
  const uint64_t nw = (d + 31) / 32;
  uint64_t pos = 0;
  auto put = [&](int i, uint64_t count, uint64_t elem) {
    L->off[i] = pos;
    L->count[i] = count;
    pos = round16(pos + count * elem);
  };
  switch (q.op) {
    case DS_Q_IDENTITY: put(0, d, 4); break;
    case DS_Q_SIGN1: put(0, nw, 4); put(1, q.chunk ? (d + q.chunk - 1) / q.chunk : 1, 4); break;
    case DS_Q_TERNARY: put(0, nw, 4); put(1, nw, 4); put(2, 1, 4); break;
    case DS_Q_TOPK: put(0, q.k, 4); put(1, q.k, 4); break;
    case DS_Q_QSGD: put(0, d, 1); put(1, nw, 4); put(2, (d + q.chunk - 1) / q.chunk, 4); break;
    case DS_Q_CLIP: put(0, d, (32 - q.levels) / 8); break;
    case DS_Q_RSPARSE: put(0, (d + q.chunk - 1) / q.chunk * (q.chunk / q.levels), 4); put(1, (d + q.chunk - 1) / q.chunk, 4); break;
  }
  L->stride = pos ? pos : 16;
}

}  // namespace

struct ds_ctx {
  ds_config cfg;
  ds_buffers buf;
  ds_payload_layout wl, sl;
  TopkPlan wplan, splan;  // workspace carving of the top-k path (worker rows / server row)
  float* acc;             // dense accumulator for sparse worker payloads (inside workspace), or NULL
  uint32_t* acc_offsets;  // span offsets of the sparse payloads (inside workspace), or NULL
  void* whole;            // scratch of the operators with one factor per vector (inside workspace), or NULL
  int phase;              // 0: step complete, 1: worker pass done, 2: unfused server pass done
  bool offsets_ready;     // the worker pass that just ran left the span table of its sparse payloads in acc_offsets
};

namespace {

// Workspace = [top-k scratch shared by both passes][dense accumulator for sparse worker payloads]
//             [threshold history of the n worker vectors][threshold history of the server vector]
// Only the histories carry meaning from one call to the next, and only as a hint.
uint64_t plan_workspace(ds_ctx* c) {
  const ds_config& cfg = c->cfg;
  uint64_t topk_bytes = 0;
  if (cfg.worker_q.op == DS_Q_TOPK) {
    topk_plan(cfg.d, cfg.n, cfg.worker_q.k, true, &c->wplan);
    topk_bytes = c->wplan.bytes;
  }
  if (cfg.server_q.op == DS_Q_TOPK) {
    topk_plan(cfg.d, 1, cfg.server_q.k, true, &c->splan);
    if (c->splan.bytes > topk_bytes) topk_bytes = c->splan.bytes;
  }
  uint64_t total = round16(topk_bytes);
  const uint64_t acc_off = total;
  if (cfg.worker_q.op == DS_Q_TOPK) total += round16(cfg.d * 4);
  const uint64_t accoff_off = total;
  if (cfg.worker_q.op == DS_Q_TOPK) total += round16(sparse_offsets_bytes(cfg.n, cfg.d));
  c->acc = (cfg.worker_q.op == DS_Q_TOPK && c->buf.workspace)
               ? reinterpret_cast<float*>(static_cast<uint8_t*>(c->buf.workspace) + acc_off)
               : nullptr;
  c->acc_offsets = (cfg.worker_q.op == DS_Q_TOPK && c->buf.workspace)
                       ? reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(c->buf.workspace) + accoff_off)
                       : nullptr;
  uint8_t* ws = static_cast<uint8_t*>(c->buf.workspace);
  if (cfg.worker_q.op == DS_Q_TOPK) {
    c->wplan.pred = ws ? reinterpret_cast<TopkPred*>(ws + total) : nullptr;
    total += round16((uint64_t)cfg.n * sizeof(TopkPred));
  }
  if (cfg.server_q.op == DS_Q_TOPK) {
    c->splan.pred = ws ? reinterpret_cast<TopkPred*>(ws + total) : nullptr;
    total += round16(sizeof(TopkPred));
  }
  // tile sums of the operators with one factor per vector (the two passes run one after the other)
  uint64_t whole_bytes = 0;
  if (whole_vector(cfg.worker_q)) whole_bytes = whole_workspace_bytes(cfg.d, cfg.n);
  if (whole_vector(cfg.server_q) && whole_workspace_bytes(cfg.d, 1) > whole_bytes) whole_bytes = whole_workspace_bytes(cfg.d, 1);
  c->whole = (whole_bytes && ws) ? ws + total : nullptr;
  total += round16(whole_bytes);
  return total;
}

SrcParams worker_src(const ds_ctx* c, const float* g) {
  SrcParams s;
  memset(&s, 0, sizeof s);
  s.g = g;
  s.delta = no_compensation(c->cfg) ? nullptr : c->buf.delta_w;
  s.d = c->cfg.d;
  s.n = c->cfg.n;
  s.vec = (c->cfg.d % 4 == 0) && aligned16(g);
  return s;
}

SrcParams server_src(const ds_ctx* c, int* kind) {
  SrcParams s;
  memset(&s, 0, sizeof s);
  const ds_qspec& wq = c->cfg.worker_q;
  s.delta = no_compensation(c->cfg) ? nullptr : c->buf.delta_s;   // NULL: v is the plain mean
  s.d = c->cfg.d;
  s.n = c->cfg.n;
  s.inv_n = 1.0f / (float)c->cfg.n;
  s.wp = static_cast<const uint8_t*>(c->buf.worker_payload);
  s.wp_stride = c->wl.stride;
  for (int i = 0; i < 3; ++i) s.wp_off[i] = c->wl.off[i];
  s.w_log2_chunk = (wq.op == DS_Q_SIGN1 || wq.op == DS_Q_QSGD || wq.op == DS_Q_RSPARSE) ? log2u(wq.chunk) : 0;
  if (whole_vector(wq)) s.w_log2_chunk = 32;   // every entry (d < 2^32) reads factor number 0
  s.w_log2_keep = wq.op == DS_Q_RSPARSE ? log2u(wq.levels) : 0;
  s.w_levels = (float)wq.levels;
  s.w_clip_bits = wq.op == DS_Q_CLIP ? wq.levels : 0;
  s.acc = c->acc;
  s.vec = 1;
  switch (wq.op) {
    case DS_Q_IDENTITY: *kind = SRC_SRV_IDENTITY; break;
    case DS_Q_SIGN1: *kind = SRC_SRV_SIGN1; break;
    case DS_Q_TOPK: *kind = SRC_SRV_TOPK; break;
    case DS_Q_CLIP: *kind = SRC_SRV_CLIP; break;
    case DS_Q_RSPARSE: *kind = SRC_SRV_RSPARSE; break;
    case DS_Q_TERNARY: *kind = SRC_SRV_TERNARY; break;
    default: *kind = SRC_SRV_QSGD; break;
  }
  return s;
}

// One compression pass over `rows` vectors: rows = n with the worker source, 1 with a server source.
// Where a pass sits inside the whole problem: d_pass entries per vector starting at entry lo of every
// row, first worker row0.  The whole-vector calls use {cfg.d, 0, 0}.
struct PassWindow {
  uint64_t d_pass, lo;
  uint32_t row0;
};

int run_pass(ds_ctx* c, int src_kind, const SrcParams& src, const ds_qspec& q, const ds_payload_layout& L,
             uint8_t* payload, float* delta, uint32_t rows, bool server, float* x_fused, uint32_t step,
             cudaStream_t st, const PassWindow* win = nullptr) {
  // a slice pass sees vectors of d_pass entries; pointers arrive already shifted to the slice, and
  // rows stay cfg.d entries apart
  const uint64_t d = win ? win->d_pass : c->cfg.d;
  const uint64_t row_stride = c->cfg.d;
  const uint64_t lo = win ? win->lo : 0;
  cudaError_t e = cudaSuccess;
  switch (q.op) {
    case DS_Q_IDENTITY:
      e = launch_identity(src_kind, src, reinterpret_cast<float*>(payload + L.off[0]) + lo, L.stride / 4, delta, row_stride,
                          x_fused, c->cfg.gamma, rows, st);
      break;
    case DS_Q_TERNARY:
    case DS_Q_SIGN1:
      if (whole_vector(q)) {
        if (win) return DS_ERR_UNSUPPORTED;
        WholeParams wp;
        memset(&wp, 0, sizeof wp);
        wp.out_sgn = reinterpret_cast<uint32_t*>(payload + L.off[0]);
        wp.out_nz = q.op == DS_Q_TERNARY ? reinterpret_cast<uint32_t*>(payload + L.off[1]) : nullptr;
        wp.out_scale = reinterpret_cast<float*>(payload + L.off[q.op == DS_Q_TERNARY ? 2 : 1]);
        wp.word_stride = L.stride / 4;
        wp.delta_out = delta;
        wp.delta_row_stride = row_stride;
        wp.x = x_fused;
        wp.gamma = c->cfg.gamma;
        wp.keys = philox_key_schedule((uint32_t)(c->cfg.seed & 0xFFFFFFFFu), (uint32_t)(c->cfg.seed >> 32));
        wp.step = step;
        wp.server_pass = server ? 1u : 0u;
        wp.l2 = (q.op == DS_Q_SIGN1 && q.norm == DS_NORM_L2) ? 1u : 0u;
        e = launch_whole(q.op, src_kind, src, wp, c->whole, rows, st);
        break;
      }
      // fall through: the 1-bit operator with a factor per chunk
    case DS_Q_QSGD: {
      ChunkParams p;
      memset(&p, 0, sizeof p);
      if (q.op == DS_Q_SIGN1) {
        p.out_bits = reinterpret_cast<uint32_t*>(payload + L.off[0]) + lo / 32;
        p.out_scale = reinterpret_cast<float*>(payload + L.off[1]) + lo / q.chunk;
      } else {
        p.out_lvl = payload + L.off[0] + lo;
        p.out_bits = reinterpret_cast<uint32_t*>(payload + L.off[1]) + lo / 32;
        p.out_scale = reinterpret_cast<float*>(payload + L.off[2]) + lo / q.chunk;
      }
      p.chunk0 = (uint32_t)(lo / q.chunk);
      p.row0 = win ? win->row0 : 0;
      p.bits_stride = L.stride / 4;
      p.scale_stride = L.stride / 4;
      p.lvl_stride = L.stride;
      p.delta_out = delta;
      p.delta_row_stride = row_stride;
      p.x = x_fused;
      p.gamma = c->cfg.gamma;
      p.levels_f = (float)q.levels;
      p.levels_u = q.levels;
      p.sign_l2 = (q.op == DS_Q_SIGN1 && q.norm == DS_NORM_L2) ? 1u : 0u;
      p.keys = philox_key_schedule((uint32_t)(c->cfg.seed & 0xFFFFFFFFu), (uint32_t)(c->cfg.seed >> 32));
      p.step = step;
      p.server_pass = server ? 1u : 0u;
      e = launch_chunked(q.op, src_kind, src, p, rows, q.chunk, st);
      break;
    }
    case DS_Q_TOPK: {
      if (win) return DS_ERR_UNSUPPORTED;
      TopkIO io;
      io.idx = reinterpret_cast<uint32_t*>(payload + L.off[0]);
      io.val = reinterpret_cast<float*>(payload + L.off[1]);
      io.payload_stride = L.stride;
      io.v_inout = delta;  // v is written over delta, then the kept entries are zeroed: delta = v - Q[v]
      io.keep_error = 1;
      // the whole-vector worker pass hands the server the span table of its index lists
      io.span_off = (!server && !win && q.k > 0) ? c->acc_offsets : nullptr;
      if (src_kind == SRC_WORKER_PLAIN) {
        // no error is kept: v is the gradient itself, selected where it lies and never written
        if (q.k == 0) return DS_OK;  // nothing to send, nothing to keep
        io.v_inout = const_cast<float*>(src.g);
        io.keep_error = 0;
      }
      io.x = x_fused;
      io.gamma = c->cfg.gamma;
      io.dev_status = c->buf.dev_status;
      e = launch_topk(src_kind, src, server ? c->splan : c->wplan, c->buf.workspace, io, rows, q.k, st);
      break;
    }
    case DS_Q_CLIP:
      e = launch_clip(src_kind, src, q.levels, payload + L.off[0] + lo * ((32 - q.levels) / 8), L.stride, delta, row_stride,
                      x_fused, c->cfg.gamma, rows, st);
      break;
    case DS_Q_RSPARSE: {
      RsparseParams rp;
      memset(&rp, 0, sizeof rp);
      rp.out_val = reinterpret_cast<float*>(payload + L.off[0]) + lo / q.levels;     // slot j / S
      rp.out_off = reinterpret_cast<uint32_t*>(payload + L.off[1]) + lo / q.chunk;
      rp.chunk0 = (uint32_t)(lo / q.chunk);
      rp.row0 = win ? win->row0 : 0;
      rp.val_stride = L.stride / 4;
      rp.off_stride = L.stride / 4;
      rp.log2_chunk = log2u(q.chunk);
      rp.log2_keep = log2u(q.levels);
      rp.scaled = q.norm == DS_RSPARSE_SCALED ? 1u : 0u;
      rp.keys = philox_key_schedule((uint32_t)(c->cfg.seed & 0xFFFFFFFFu), (uint32_t)(c->cfg.seed >> 32));
      rp.step = step;
      rp.server_pass = server ? 1u : 0u;
      e = launch_rsparse(src_kind, src, rp, delta, row_stride, x_fused, c->cfg.gamma, rows, st);
      break;
    }
    default: return DS_ERR_UNSUPPORTED;
  }
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "kernel launch");
}

}  // namespace

extern "C" {

int ds_version(void) { return 100; }

uint64_t ds_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

const char* ds_last_error(void) { return g_last_error; }

int ds_get_layout(const ds_config* cfg, int which, ds_payload_layout* out) {
  if (!config_ok(cfg) || !out || (which != 0 && which != 1)) return DS_ERR_INVALID_ARG;
  layout_of(which == 0 ? cfg->worker_q : cfg->server_q, cfg->d, out);
  return DS_OK;
}

int ds_create(const ds_config* cfg, ds_buffers* bufs, ds_handle* out) {
  if (!config_ok(cfg) || !bufs) return DS_ERR_INVALID_ARG;
  ds_ctx tmp;
  memset(&tmp, 0, sizeof tmp);
  tmp.cfg = *cfg;
  tmp.buf = *bufs;
  layout_of(cfg->worker_q, cfg->d, &tmp.wl);
  layout_of(cfg->server_q, cfg->d, &tmp.sl);
  // without compensation no error is carried: delta_w is not needed at all, delta_s only as the place
  // where a top-k server pass lays out its vector
  const bool nocomp = no_compensation(*cfg);
  const uint64_t need_x = cfg->d * 4, need_dw = nocomp ? 0 : (uint64_t)delta_rows(*cfg) * cfg->d * 4;
  const uint64_t need_ds = (nocomp && cfg->server_q.op != DS_Q_TOPK) ? 0 : cfg->d * 4;
  const uint64_t need_wp = (uint64_t)cfg->n * tmp.wl.stride, need_sp = tmp.sl.stride;
  const uint64_t need_ws = plan_workspace(&tmp);
  if (bufs->x == nullptr) {  // query mode
    bufs->x_bytes = need_x;
    bufs->delta_w_bytes = need_dw;
    bufs->delta_s_bytes = need_ds;
    bufs->worker_payload_bytes = need_wp;
    bufs->server_payload_bytes = need_sp;
    bufs->workspace_bytes = need_ws;
    return DS_NEED_BUFFERS;
  }
  if (!out) return DS_ERR_INVALID_ARG;
  if ((need_dw && !bufs->delta_w) || (need_ds && !bufs->delta_s) || !bufs->worker_payload || !bufs->server_payload ||
      !bufs->dev_status)
    return DS_ERR_INVALID_ARG;
  if (need_ws && !bufs->workspace) return DS_ERR_INVALID_ARG;
  const void* ptrs[] = {bufs->x, bufs->delta_w, bufs->delta_s, bufs->worker_payload, bufs->server_payload, bufs->workspace};
  for (const void* p : ptrs)
    if (!aligned16(p)) return DS_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(bufs->dev_status) & 3u) != 0) return DS_ERR_ALIGN;
  if (bufs->x_bytes < need_x || bufs->delta_w_bytes < need_dw || bufs->delta_s_bytes < need_ds ||
      bufs->worker_payload_bytes < need_wp || bufs->server_payload_bytes < need_sp || bufs->workspace_bytes < need_ws)
    return DS_ERR_BUFFER_TOO_SMALL;
  ds_ctx* c = new (std::nothrow) ds_ctx(tmp);
  if (!c) return DS_ERR_INVALID_ARG;
  plan_workspace(c);
  c->phase = 0;
  *out = c;
  return DS_OK;
}

int ds_worker_compress(ds_handle h, const float* g, uint32_t step, void* cuda_stream) {
  if (!h || !g) return DS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(g) & 3u) != 0) return DS_ERR_ALIGN;
  if (h->phase != 0) return DS_ERR_STATE;
  if (delta_rows(h->cfg) != h->cfg.n) return DS_ERR_UNSUPPORTED;   // this instance holds the errors of one block of workers only
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const SrcParams src = worker_src(h, g);
  const bool nocomp = no_compensation(h->cfg);
  const int rc = run_pass(h, nocomp ? SRC_WORKER_PLAIN : SRC_WORKER, src, h->cfg.worker_q, h->wl,
                          static_cast<uint8_t*>(h->buf.worker_payload), nocomp ? nullptr : h->buf.delta_w, h->cfg.n, false,
                          nullptr, step, st);
  if (rc == DS_OK) {
    h->phase = 1;
    h->offsets_ready = h->cfg.worker_q.op == DS_Q_TOPK && h->cfg.worker_q.k > 0;
  }
  return rc;
}

int ds_server_aggregate_compress(ds_handle h, uint32_t step, uint32_t flags, void* cuda_stream) {
  if (!h || (flags & ~DS_FUSE_APPLY)) return DS_ERR_INVALID_ARG;
  if (h->phase != 1) return DS_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int kind = 0;
  const SrcParams src = server_src(h, &kind);
  if (kind == SRC_SRV_TOPK) {
    // (1/n) sum_i Q[v_i] for sparse payloads: dense accumulator, workers added in order 0..n-1
    const cudaError_t e = launch_sparse_accumulate(static_cast<const uint8_t*>(h->buf.worker_payload), h->wl.stride,
                                                   h->wl.off[0], h->wl.off[1], h->cfg.n, h->cfg.worker_q.k, h->cfg.d,
                                                   h->acc_offsets, h->offsets_ready, h->acc, st);
    h->offsets_ready = false;
    if (e != cudaSuccess) return cuda_fail(e, "sparse accumulate");
  }
  const bool fuse = (flags & DS_FUSE_APPLY) != 0;
  // without compensation the residual has no destination -- except that a top-k pass still lays its
  // vector out in delta_s (which is then scratch: never read back)
  float* ds_out = (no_compensation(h->cfg) && h->cfg.server_q.op != DS_Q_TOPK) ? nullptr : h->buf.delta_s;
  const int rc = run_pass(h, kind, src, h->cfg.server_q, h->sl, static_cast<uint8_t*>(h->buf.server_payload), ds_out, 1, true,
                          fuse ? h->buf.x : nullptr, step, st);
  if (rc == DS_OK) h->phase = fuse ? 0 : 2;
  return rc;
}

int ds_apply_update(ds_handle h, void* cuda_stream) {
  if (!h) return DS_ERR_INVALID_ARG;
  if (h->phase != 2) return DS_ERR_STATE;
  const ds_qspec& q = h->cfg.server_q;
  PayloadView pv;
  memset(&pv, 0, sizeof pv);
  pv.op = q.op;
  pv.base = static_cast<const uint8_t*>(h->buf.server_payload);
  for (int i = 0; i < 3; ++i) pv.off[i] = h->sl.off[i];
  pv.log2_chunk = (q.op == DS_Q_SIGN1 || q.op == DS_Q_QSGD || q.op == DS_Q_RSPARSE) ? log2u(q.chunk) : 0;
  if (whole_vector(q)) pv.log2_chunk = 32;   // one factor: every entry reads number 0
  pv.levels_f = (float)q.levels;
  pv.clip_bits = q.op == DS_Q_CLIP ? q.levels : 0;
  pv.log2_keep = q.op == DS_Q_RSPARSE ? log2u(q.levels) : 0;
  pv.k = q.k;
  const cudaError_t e = launch_apply(pv, h->buf.x, h->cfg.d, h->cfg.gamma, static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(e, "apply update");
  h->phase = 0;
  return DS_OK;
}

namespace {

bool slice_ok(const ds_ctx* h, uint64_t lo, uint64_t hi) {
  const uint64_t d = h->cfg.d;
  return lo < hi && hi <= d && lo % DS_SLICE_ALIGN == 0 && (hi == d || hi % DS_SLICE_ALIGN == 0);
}

bool sliceable(const ds_qspec& q) { return q.op != DS_Q_TOPK && !whole_vector(q); }

}  // namespace

int ds_worker_compress_rows(ds_handle h, const float* g, uint32_t row0, uint32_t nrows, uint32_t step, void* cuda_stream) {
  if (!h || !g || nrows == 0 || (uint64_t)row0 + nrows > h->cfg.n) return DS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(g) & 3u) != 0) return DS_ERR_ALIGN;
  if (!sliceable(h->cfg.worker_q)) return DS_ERR_UNSUPPORTED;
  const uint64_t d = h->cfg.d;
  SrcParams src = worker_src(h, g);
  const bool nocomp = no_compensation(h->cfg);
  // with the errors of one block of R workers only, worker i lives in row i mod R and a call stays inside a block
  const uint32_t R = delta_rows(h->cfg);
  if ((uint64_t)(row0 % R) + nrows > R) return DS_ERR_INVALID_ARG;
  float* delta_blk = nocomp ? nullptr : h->buf.delta_w + (uint64_t)(row0 % R) * d;
  src.delta = delta_blk;
  src.vec = (d % 4 == 0) && aligned16(g);
  const PassWindow win{d, 0, row0};
  return run_pass(h, nocomp ? SRC_WORKER_PLAIN : SRC_WORKER, src, h->cfg.worker_q, h->wl,
                  static_cast<uint8_t*>(h->buf.worker_payload) + (uint64_t)row0 * h->wl.stride, delta_blk, nrows, false, nullptr,
                  step, static_cast<cudaStream_t>(cuda_stream), &win);
}

int ds_server_aggregate_compress_slice(ds_handle h, uint32_t step, uint32_t flags, uint64_t lo, uint64_t hi,
                                       void* cuda_stream) {
  if (!h || (flags & ~DS_FUSE_APPLY) || !slice_ok(h, lo, hi)) return DS_ERR_INVALID_ARG;
  if (!sliceable(h->cfg.worker_q) || !sliceable(h->cfg.server_q)) return DS_ERR_UNSUPPORTED;
  int kind = 0;
  SrcParams src = server_src(h, &kind);
  const ds_qspec& wq = h->cfg.worker_q;
  // the slice of every worker payload: shift each sub-array to entry lo
  src.d = hi - lo;
  float* ds_slice = no_compensation(h->cfg) ? nullptr : h->buf.delta_s + lo;
  src.delta = ds_slice;
  switch (wq.op) {
    case DS_Q_IDENTITY: src.wp_off[0] += lo * 4; break;
    case DS_Q_SIGN1: src.wp_off[0] += lo / 8; src.wp_off[1] += lo / wq.chunk * 4; break;
    case DS_Q_QSGD: src.wp_off[0] += lo; src.wp_off[1] += lo / 8; src.wp_off[2] += lo / wq.chunk * 4; break;
    case DS_Q_CLIP: src.wp_off[0] += lo * ((32 - wq.levels) / 8); break;
    case DS_Q_RSPARSE: src.wp_off[0] += lo / wq.levels * 4; src.wp_off[1] += lo / wq.chunk * 4; break;
    default: return DS_ERR_UNSUPPORTED;
  }
  const PassWindow win{hi - lo, lo, 0};
  const bool fuse = (flags & DS_FUSE_APPLY) != 0;
  return run_pass(h, kind, src, h->cfg.server_q, h->sl, static_cast<uint8_t*>(h->buf.server_payload), ds_slice, 1,
                  true, fuse ? h->buf.x + lo : nullptr, step, static_cast<cudaStream_t>(cuda_stream), &win);
}

int ds_apply_update_slice(ds_handle h, uint64_t lo, uint64_t hi, void* cuda_stream) {
  if (!h || !slice_ok(h, lo, hi)) return DS_ERR_INVALID_ARG;
  const ds_qspec& q = h->cfg.server_q;
  if (!sliceable(q)) return DS_ERR_UNSUPPORTED;
  PayloadView pv;
  memset(&pv, 0, sizeof pv);
  pv.op = q.op;
  pv.base = static_cast<const uint8_t*>(h->buf.server_payload);
  for (int i = 0; i < 3; ++i) pv.off[i] = h->sl.off[i];
  pv.log2_chunk = (q.op == DS_Q_SIGN1 || q.op == DS_Q_QSGD || q.op == DS_Q_RSPARSE) ? log2u(q.chunk) : 0;
  pv.levels_f = (float)q.levels;
  pv.clip_bits = q.op == DS_Q_CLIP ? q.levels : 0;
  pv.log2_keep = q.op == DS_Q_RSPARSE ? log2u(q.levels) : 0;
  switch (q.op) {
    case DS_Q_IDENTITY: pv.off[0] += lo * 4; break;
    case DS_Q_SIGN1: pv.off[0] += lo / 8; pv.off[1] += lo / q.chunk * 4; break;
    case DS_Q_QSGD: pv.off[0] += lo; pv.off[1] += lo / 8; pv.off[2] += lo / q.chunk * 4; break;
    case DS_Q_CLIP: pv.off[0] += lo * ((32 - q.levels) / 8); break;
    case DS_Q_RSPARSE: pv.off[0] += lo / q.levels * 4; pv.off[1] += lo / q.chunk * 4; break;
    default: return DS_ERR_UNSUPPORTED;
  }
  const cudaError_t e = launch_apply(pv, h->buf.x + lo, hi - lo, h->cfg.gamma, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "apply update");
}

// ---- global top-k on the server pass when the vector's slices live on different GPUs ----------

namespace {
bool topk_slice_ok(const ds_ctx* h, uint64_t lo, uint64_t hi) {
  return h->cfg.server_q.op == DS_Q_TOPK && h->cfg.server_q.k > 0 && sliceable(h->cfg.worker_q) && slice_ok(h, lo, hi);
}
}  // namespace

int ds_server_topk_slice_begin(ds_handle h, uint32_t step, uint64_t lo, uint64_t hi, uint32_t* hist, void* cuda_stream) {
  (void)step;   // the selection draws nothing
  if (!h || !hist || (reinterpret_cast<uintptr_t>(hist) & 15u)) return DS_ERR_INVALID_ARG;
  if (h->cfg.server_q.op != DS_Q_TOPK || !sliceable(h->cfg.worker_q)) return DS_ERR_UNSUPPORTED;
  if (!topk_slice_ok(h, lo, hi)) return DS_ERR_INVALID_ARG;
  int kind = 0;
  SrcParams src = server_src(h, &kind);
  const ds_qspec& wq = h->cfg.worker_q;
  src.d = hi - lo;
  float* ds_slice = h->buf.delta_s + lo;   // v is laid out here; without compensation it is scratch
  src.delta = no_compensation(h->cfg) ? nullptr : ds_slice;
  switch (wq.op) {
    case DS_Q_IDENTITY: src.wp_off[0] += lo * 4; break;
    case DS_Q_SIGN1: src.wp_off[0] += lo / 8; src.wp_off[1] += lo / wq.chunk * 4; break;
    case DS_Q_QSGD: src.wp_off[0] += lo; src.wp_off[1] += lo / 8; src.wp_off[2] += lo / wq.chunk * 4; break;
    case DS_Q_CLIP: src.wp_off[0] += lo * ((32 - wq.levels) / 8); break;
    case DS_Q_RSPARSE: src.wp_off[0] += lo / wq.levels * 4; src.wp_off[1] += lo / wq.chunk * 4; break;
    default: return DS_ERR_UNSUPPORTED;
  }
  const cudaError_t e = launch_topk_slice_begin(kind, src, h->buf.workspace, ds_slice, h->cfg.server_q.k, hist,
                                                static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "top-k over a slice, first histogram");
}

int ds_server_topk_slice_digit(ds_handle h, int level, uint64_t lo, uint64_t hi, uint32_t* hist_sum, uint32_t* hist_next,
                               void* cuda_stream) {
  if (!h || !hist_sum || !hist_next || level < 1 || level > 3) return DS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(hist_sum) | reinterpret_cast<uintptr_t>(hist_next)) & 15u) return DS_ERR_ALIGN;
  if (h->cfg.server_q.op != DS_Q_TOPK) return DS_ERR_UNSUPPORTED;
  if (!topk_slice_ok(h, lo, hi)) return DS_ERR_INVALID_ARG;
  const cudaError_t e = launch_topk_slice_digit(level, h->buf.workspace, h->buf.delta_s + lo, hi - lo, 1, h->cfg.server_q.k, hist_sum,
                                                hist_next, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "top-k over a slice, digit");
}

int ds_server_topk_slice_emit(ds_handle h, uint64_t lo, uint64_t hi, uint32_t ties_to_keep, uint32_t count, uint64_t first_slot,
                              uint32_t flags, void* cuda_stream) {
  if (!h || (flags & ~DS_FUSE_APPLY)) return DS_ERR_INVALID_ARG;
  if (h->cfg.server_q.op != DS_Q_TOPK) return DS_ERR_UNSUPPORTED;
  if (!topk_slice_ok(h, lo, hi) || first_slot + count > h->cfg.server_q.k) return DS_ERR_INVALID_ARG;
  uint8_t* sp = static_cast<uint8_t*>(h->buf.server_payload);
  uint32_t* idx = reinterpret_cast<uint32_t*>(sp + h->sl.off[0]) + first_slot;
  float* val = reinterpret_cast<float*>(sp + h->sl.off[1]) + first_slot;
  const cudaError_t e = launch_topk_slice_emit(h->buf.workspace, h->buf.delta_s + lo, hi - lo, h->cfg.server_q.k, ties_to_keep, count,
                                               (uint32_t)lo, idx, val, (flags & DS_FUSE_APPLY) ? h->buf.x + lo : nullptr, h->cfg.gamma,
                                               static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "top-k over a slice, emit");
}

int ds_apply_update_sparse_range(ds_handle h, uint64_t first_slot, uint64_t count, void* cuda_stream) {
  if (!h) return DS_ERR_INVALID_ARG;
  if (h->cfg.server_q.op != DS_Q_TOPK) return DS_ERR_UNSUPPORTED;
  if (first_slot + count > h->cfg.server_q.k) return DS_ERR_INVALID_ARG;
  if (count == 0) return DS_OK;
  PayloadView pv;
  memset(&pv, 0, sizeof pv);
  pv.op = DS_Q_TOPK;
  pv.base = static_cast<const uint8_t*>(h->buf.server_payload);
  pv.off[0] = h->sl.off[0] + first_slot * 4;
  pv.off[1] = h->sl.off[1] + first_slot * 4;
  pv.k = count;
  const cudaError_t e = launch_apply(pv, h->buf.x, h->cfg.d, h->cfg.gamma, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "apply update, part of a sparse payload");
}

int ds_step_host(ds_handle h, const float* g_host, float* g_dev, uint32_t step, void* server_payload_host, float* x_host,
                 void* cuda_stream) {
  if (!h || !g_host || !g_dev) return DS_ERR_INVALID_ARG;
  if (!aligned16(g_dev)) return DS_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(g_dev, g_host, (uint64_t)h->cfg.n * h->cfg.d * 4, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(e, "copy of g to the device");
  int rc = ds_worker_compress(h, g_dev, step, cuda_stream);
  if (rc != DS_OK) return rc;
  rc = ds_server_aggregate_compress(h, step, DS_FUSE_APPLY, cuda_stream);
  if (rc != DS_OK) return rc;
  if (server_payload_host) {
    e = cudaMemcpyAsync(server_payload_host, h->buf.server_payload, h->sl.stride, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "copy of the server payload to the host");
  }
  if (x_host) {
    e = cudaMemcpyAsync(x_host, h->buf.x, h->cfg.d * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "copy of x to the host");
  }
  return DS_OK;
}

int ds_destroy(ds_handle h) {
  if (!h) return DS_ERR_INVALID_ARG;
  delete h;
  return DS_OK;
}

}  // extern "C"
