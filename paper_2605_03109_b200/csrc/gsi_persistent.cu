// Host entry points of the persistent decode-step kernel, its small helper kernels, and
// the build of the kernel for stacks without concurrent groups.
#include <cuda_fp8.h>

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
    // within a tile: four 8 x 8 blocks of 128 bytes, each row-major with 16-byte rows
    const int blk = (int)((wi >> 5) & 3), g = (int)((wi >> 2) & 7), t = (int)(wi & 3);
    const size_t tile = wi >> 7;
    const int K = (int)(tile % kt);
    const size_t R = tile / kt;
    const size_t row = R * 16 + g + (blk & 1) * 8;
    const int col = K * 16 + 2 * t + (blk >> 1) * 8;
    dst[wi] = row < (size_t)rows ? *reinterpret_cast<const uint32_t*>(src + row * k + col) : 0u;
  }
}

// The image in FP8 (Section 7.4): one block per 16 rows.  Row scale = max|row| / 448 (1 for a
// zero row), code = nearest E4M3 of element / scale (ties to even, saturating); both
// divisions are single IEEE fp32 operations, so the codes follow from the bf16 image alone.
__global__ void k_pack_t16_fp8(const uint16_t* __restrict__ src, int rows, int k, unsigned char* __restrict__ dst) {
  __shared__ float s_scale[16];
  const int kt = k >> 4;
  const size_t R = blockIdx.x;
  const int tid = threadIdx.x;
  {
    const int row = tid >> 4, sub = tid & 15;
    float amax = 0.f;
    if (R * 16 + row < (size_t)rows)
      for (int j = sub; j < k; j += 16)
        amax = fmaxf(amax, fabsf(__uint_as_float((uint32_t)src[(R * 16 + row) * k + j] << 16)));
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (sub == 0) s_scale[row] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
  }
  __syncthreads();
  unsigned char* out = dst + R * (size_t)persist_image_row_bytes(k, true);
  for (int wi = tid; wi < kt * 128; wi += blockDim.x) {   // one pair of codes per step
    const int reg = wi & 3, lane = (wi >> 2) & 31, K = wi >> 7;
    const int g = lane >> 2, t = lane & 3;
    const int r16 = g + (reg & 1) * 8;
    const size_t row = R * 16 + r16;
    const int col = K * 16 + 2 * t + (reg >> 1) * 8;
    unsigned short pair = 0;
    if (row < (size_t)rows) {
      const float sc = s_scale[r16];
      const float a = __uint_as_float((uint32_t)src[row * k + col] << 16);
      const float b = __uint_as_float((uint32_t)src[row * k + col + 1] << 16);
      const unsigned lo = __nv_cvt_float_to_fp8(__fdiv_rn(a, sc), __NV_SATFINITE, __NV_E4M3);
      const unsigned hi = __nv_cvt_float_to_fp8(__fdiv_rn(b, sc), __NV_SATFINITE, __NV_E4M3);
      pair = (unsigned short)(lo | (hi << 8));
    }
    reinterpret_cast<unsigned short*>(out)[wi] = pair;
  }
  if (tid < 16) reinterpret_cast<float*>(out + (size_t)kt * 256)[tid] = s_scale[tid];
}

}  // namespace

cudaError_t launch_pack_t16_fp8(const void* src, int rows, int k, void* dst, cudaStream_t st) {
  k_pack_t16_fp8<<<(rows + 15) / 16, 256, 0, st>>>(static_cast<const uint16_t*>(src), rows, k,
                                                  static_cast<unsigned char*>(dst));
  return cudaGetLastError();
}

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
