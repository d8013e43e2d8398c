// Host entry points of the persistent decode-step kernel, its small helper kernels, and
// the build of the kernel for stacks without concurrent groups.
#include "gsi_persistent_impl.cuh"

namespace gsi {

namespace {

__global__ void k_abs_max_bf16(const uint16_t* __restrict__ p, size_t n, float* out) {
  // max |P|, written as a float; the values are non-negative so the integer
  // ordering of their bit patterns is the numeric ordering.
  float m = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x) {
    const float v = fabsf(__uint_as_float(((uint32_t)p[i]) << 16));
    m = fmaxf(m, v);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
}

__global__ void k_patch_pmax(PersistGroup* groups, const float* const* pmax_ptrs, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n && pmax_ptrs[i]) groups[i].pmax = *pmax_ptrs[i];
}

}  // namespace

cudaError_t launch_patch_pmax(PersistGroup* groups, const float* const* pmax_ptrs, int n,
                              cudaStream_t st) {
  k_patch_pmax<<<(n + 127) / 128, 128, 0, st>>>(groups, pmax_ptrs, n);
  return cudaGetLastError();
}

int persist_smem_bytes() { return kSmemBytes; }
int persist_threads() { return kThreadsP; }

cudaError_t launch_abs_max_bf16(const void* p, size_t n, float* out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
  if (e != cudaSuccess) return e;
  k_abs_max_bf16<<<64, 256, 0, st>>>(static_cast<const uint16_t*>(p), n, out);
  return cudaGetLastError();
}

// the other builds of the kernel live in translation units of their own
cudaError_t launch_decode_step_pairs(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_k128(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_pairs_k128(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_k256(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_pairs_k256(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_k512(const PersistParams& p, int grid, cudaStream_t st);
cudaError_t launch_decode_step_pairs_k512(const PersistParams& p, int grid, cudaStream_t st);

cudaError_t launch_decode_step(const PersistParams& p, int grid, bool pairs, int common_k,
                               cudaStream_t st) {
  switch (common_k) {
    case 128:
      return pairs ? launch_decode_step_pairs_k128(p, grid, st) : launch_decode_step_k128(p, grid, st);
    case 256:
      return pairs ? launch_decode_step_pairs_k256(p, grid, st) : launch_decode_step_k256(p, grid, st);
    case 512:
      return pairs ? launch_decode_step_pairs_k512(p, grid, st) : launch_decode_step_k512(p, grid, st);
    default:
      return pairs ? launch_decode_step_pairs(p, grid, st) : launch_decode_step_t<false, 0>(p, grid, st);
  }
}

}  // namespace gsi
