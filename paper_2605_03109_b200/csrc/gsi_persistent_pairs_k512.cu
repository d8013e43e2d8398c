// A build of the persistent decode-step kernel (see gsi_persistent_impl.cuh):
// two independent groups may share a phase, every group of rank 512.
// A translation unit of its own: each build of the kernel is compiled separately.
#include "gsi_persistent_impl.cuh"

namespace gsi {

cudaError_t launch_decode_step_pairs_k512(const PersistParams& p, int grid, cudaStream_t st) {
  return launch_decode_step_t<true, 512>(p, grid, st);
}

}  // namespace gsi
