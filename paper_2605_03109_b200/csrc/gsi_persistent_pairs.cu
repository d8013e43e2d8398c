// The build of the persistent decode-step kernel that runs two independent groups in one
// phase (see gsi_persistent_impl.cuh).  A translation unit of its own: each build of the
// kernel is compiled separately.
#include "gsi_persistent_impl.cuh"

namespace gsi {

cudaError_t launch_decode_step_pairs(const PersistParams& p, int grid, cudaStream_t st) {
  return launch_decode_step_t<true>(p, grid, st);
}

}  // namespace gsi
