// Dispatch of the chunk-wise operators onto their kernels (dsq_chunked.cuh); the instantiations are
// spread over one translation unit per operator so that they compile side by side.
#include "dsq_internal.h"

namespace dsq {

cudaError_t launch_chunked_sign1(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                 cudaStream_t st);
cudaError_t launch_chunked_sign1_l2(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                    cudaStream_t st);
cudaError_t launch_chunked_qsgd_window(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                       cudaStream_t st);
cudaError_t launch_chunked_qsgd(int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                                cudaStream_t st);

cudaError_t launch_chunked(int op, int srck, const SrcParams& src, const ChunkParams& p, uint32_t rows, uint32_t chunk,
                           cudaStream_t st) {
  if (op == DS_Q_SIGN1)
    return p.sign_l2 ? launch_chunked_sign1_l2(srck, src, p, rows, chunk, st)
                     : launch_chunked_sign1(srck, src, p, rows, chunk, st);
  if (op == DS_Q_QSGD)
    return (p.chunk0 | p.row0) ? launch_chunked_qsgd_window(srck, src, p, rows, chunk, st)
                               : launch_chunked_qsgd(srck, src, p, rows, chunk, st);
  return cudaErrorInvalidValue;
}

}  // namespace dsq
