// The 1-bit operator with the scale from l2 magnitudes: instantiations of the chunk kernel.
#include "dsq_chunked.cuh"

namespace dsq {
cudaError_t launch_chunked_sign1_l2(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                    cudaStream_t st) {
  return launch_src<kOpSign1L2>(srck, src, p, rows, chunk, st);
}
}  // namespace dsq
