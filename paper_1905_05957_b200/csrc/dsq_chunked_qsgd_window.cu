// Randomised s-level quantisation over a window of the problem (some workers, or a slice of d):
// instantiations of the chunk kernel whose Philox counters carry the window's offsets.
#include "dsq_chunked.cuh"

namespace dsq {
cudaError_t launch_chunked_qsgd_window(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                       cudaStream_t st) {
  return launch_src<kOpQsgdWindow>(srck, src, p, rows, chunk, st);
}
}  // namespace dsq
