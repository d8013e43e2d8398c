// A build of the persistent decode-step kernel (see gsi_persistent_impl.cuh):
// no pairs, every group of rank 512.
// A translation unit of its own: each build of the kernel is compiled separately.
#include "gsi_persistent_impl.cuh"

namespace gsi {

cudaError_t launch_decode_step_k512(const PersistParams& p, int grid, cudaStream_t st) {
  return launch_decode_step_t<false, 512>(p, grid, st);
}

}  // namespace gsi
