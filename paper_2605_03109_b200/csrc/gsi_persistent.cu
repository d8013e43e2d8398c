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

// One thread per 32-bit word of the tiled copy.
__global__ void k_pack_t16(const uint16_t* __restrict__ src, int rows, int k, uint32_t* __restrict__ dst) {
  const int kt = k >> 4;
  const size_t n_words = (size_t)((rows + 15) / 16) * kt * 128;
  for (size_t wi = (size_t)blockIdx.x * blockDim.x + threadIdx.x; wi < n_words;
       wi += (size_t)gridDim.x * blockDim.x) {
    const int reg = (int)(wi & 3), lane = (int)((wi >> 2) & 31);
    const size_t tile = wi >> 7;
    const int K = (int)(tile % kt);
    const size_t R = tile / kt;
    const int g = lane >> 2, t = lane & 3;
    const size_t row = R * 16 + g + (reg & 1) * 8;
    const int col = K * 16 + 2 * t + (reg >> 1) * 8;
    dst[wi] = row < (size_t)rows ? *reinterpret_cast<const uint32_t*>(src + row * k + col) : 0u;
  }
}

}  // namespace

cudaError_t launch_pack_t16(const void* src, int rows, int k, void* dst, cudaStream_t st) {
  k_pack_t16<<<592, 256, 0, st>>>(static_cast<const uint16_t*>(src), rows, k, static_cast<uint32_t*>(dst));
  return cudaGetLastError();
}

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
