// Top-k with error feedback for one vector, for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc (or any allocator) at the point where they
// compress: code running inside a stream capture, a plug-in handed only its tensors by a framework
// that owns the memory pool, a real-time loop with allocation forbidden after start-up.  For them
// the radix select's scratch (histogram, select state, two selection bitmaps, segment counts) lives
// in a fixed array inside the library image instead of a caller-provided workspace.
#include <mutex>

#include "dsq_internal.h"

using namespace dsq;

namespace {

// Scratch for one selection over at most DS_STATIC_TOPK_MAX_D entries: 16 KiB histogram, a few words of
// select state, two bitmaps of MAX_D/8 bytes each and the segment counts -- about 2.03 MiB.
// Every GPU that loads the library holds this array until the process exits.
constexpr size_t kScratchBytes = 16384 + 32 + 2 * (DS_STATIC_TOPK_MAX_D / 8) + (DS_STATIC_TOPK_MAX_D / 8192) * 8 + 256;
static __device__ __align__(256) unsigned char g_topk_scratch[kScratchBytes];

// In host code g_topk_scratch is only a handle for the runtime, not a device address; the address
// that kernels may dereference is asked for once per device and remembered here.
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_topk_scratch);  // resolves the copy of the array on the current device
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int ds_topk_worker_static(const float* g, float* delta, uint64_t d, uint64_t k, uint32_t* idx, float* val,
                                     uint32_t* dev_status, void* cuda_stream) {
  if (!g || !delta || !dev_status || d < 1 || k > d || (k && (!idx || !val))) return DS_ERR_INVALID_ARG;
  if (d > DS_STATIC_TOPK_MAX_D) return DS_ERR_UNSUPPORTED;  // the fixed scratch cannot hold this selection
  const uintptr_t all = reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(delta) |
                        reinterpret_cast<uintptr_t>(idx) | reinterpret_cast<uintptr_t>(val) |
                        reinterpret_cast<uintptr_t>(dev_status);
  if (all & 3u) return DS_ERR_ALIGN;
  TopkPlan plan;
  topk_plan(d, 1, k, false, &plan);  // no candidate list: the scratch stays small
  if (plan.bytes > kScratchBytes) return DS_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  const cudaError_t es = scratch_for_current_device(&scratch);
  if (es != cudaSuccess) return cuda_fail(es, "address of the built-in top-k scratch");

  SrcParams src = {};
  src.g = g;
  src.delta = delta;
  src.d = d;
  src.n = 1;
  src.vec = (d % 4 == 0) && ((reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(delta)) & 15u) == 0;
  TopkIO io = {};
  io.idx = idx;
  io.val = val;
  io.payload_stride = 0;  // a single vector
  io.v_inout = delta;
  io.keep_error = 1;
  io.span_off = nullptr;
  io.x = nullptr;
  io.gamma = 0.f;
  io.dev_status = dev_status;
  // launch_topk clears the histogram itself; the select state, both bitmaps (whole segments) and
  // the segment counts are fully rewritten before they are read, so nothing of an earlier call
  // survives into this one.
  const cudaError_t e = launch_topk(SRC_WORKER, src, plan, scratch, io, 1, k, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? DS_OK : cuda_fail(e, "top-k with built-in scratch");
}
