// Online extension of the basis by one vector (the paper's "time-dimension tracking",
// Section 5.4, and "online basis adaptation", Section 7.2): a token is tested against
// the basis in use; if rho = ||x - P P^T x|| / ||x|| exceeds a threshold, the residual,
// orthogonalised against P twice (Gram-Schmidt with one re-orthogonalisation, "DGKS") and
// normalised, becomes column k_active of P, and W times that column (Section 4.2) becomes
// column k_active of every cached image.  Columns [k_active, k) of P are zero before, so
// every other kernel of the library keeps working on the full width k.
//
// A rare, set-up-like operation: it reuses the CUDA-core projection / residual kernels
// (twice) and the gated W r GEMV (once, for the image column) and adds three small
// kernels of its own.  Everything stays on the device: no host synchronisation.
#include "gsi_common.cuh"

namespace gsi {

namespace {

constexpr int kExtThreads = 1024;

__device__ __forceinline__ uint16_t to_bf16_bits(float v) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  return *reinterpret_cast<const uint16_t*>(&h);
}

// After the first pass: keep rho of the token (it is the quantity the threshold tests).
__global__ void k_ext_keep_rho(GroupParams g, ExtendArgs a) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    a.inv_norm[1] = g.rho_scratch[0];
    if (a.rho_out) *a.rho_out = g.rho_scratch[0];
  }
}

// After the second pass: ||r2||^2 in a fixed order, the decision, and the list of "fired"
// tokens the W r GEMV works from (token 0 if a column is appended, nobody otherwise).
__global__ void __launch_bounds__(kExtThreads) k_ext_decide(GroupParams g, ExtendArgs a) {
  __shared__ double s_part[kExtThreads / 32];
  double s = 0.0;
  for (int i = threadIdx.x; i < g.d; i += kExtThreads) s += (double)g.r[i] * (double)g.r[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kExtThreads / 32; ++w) t += s_part[w];
    const int col = *a.k_active;
    const float rho = a.inv_norm[1];
    // rho > tau is false for NaN: a non-finite token never extends the basis
    const bool go = rho > a.tau && col >= 0 && col < g.k && t > 0.0 && t < 1e300;
    a.ctrl[0] = go ? 1 : 0;
    a.ctrl[1] = col;
    a.inv_norm[0] = go ? (float)(1.0 / sqrt(t)) : 0.f;
    *g.n_fired = go ? 1 : 0;
    g.fired[0] = 0;
    if (a.appended_out) *a.appended_out = go ? 1 : 0;
  }
}

// v = r2 / ||r2|| rounded to the basis type goes into column `col` of P (and row `col` of
// the transposed copy); g.r receives the STORED value, so the image column is W times
// what the basis really holds.
__global__ void __launch_bounds__(256) k_ext_store_vector(GroupParams g, ExtendArgs a) {
  if (!a.ctrl[0]) return;
  const int col = a.ctrl[1];
  const float inv = a.inv_norm[0];
  float m = 0.f;
  for (int i = blockIdx.x * 256 + threadIdx.x; i < g.d; i += gridDim.x * 256) {
    const float v = g.r[i] * inv;
    float stored;
    if (g.p_f32) {
      const_cast<float*>(static_cast<const float*>(g.P))[(size_t)i * g.k + col] = v;
      stored = v;
    } else {
      const uint16_t b = to_bf16_bits(v);
      const_cast<uint16_t*>(static_cast<const uint16_t*>(g.P))[(size_t)i * g.k + col] = b;
      if (a.PT) a.PT[(size_t)col * g.d + i] = b;
      stored = __uint_as_float((uint32_t)b << 16);
    }
    g.r[i] = stored;
    m = fmaxf(m, fabsf(stored));
  }
  if (a.pmax) {   // max |P| of the handle: non-negative floats order like their bit patterns
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int*>(a.pmax), __float_as_int(m));
  }
}

// Column `col` of the concatenated images = bf16(W v); then the basis is one column wider.
__global__ void __launch_bounds__(256) k_ext_store_image(GroupParams g, ExtendArgs a) {
  if (!a.ctrl[0]) return;
  const int col = a.ctrl[1];
  uint16_t* WP = const_cast<uint16_t*>(g.WP);
  for (int r = blockIdx.x * 256 + threadIdx.x; r < g.O; r += gridDim.x * 256)
    WP[(size_t)r * g.k + col] = to_bf16_bits(a.y_scratch[r]);
  if (blockIdx.x == 0 && threadIdx.x == 0) *a.k_active = col + 1;
}

}  // namespace

cudaError_t launch_extend_basis(const GroupParams& g, const ExtendArgs& a, cudaStream_t st) {
  IoRef io{};
  io.x = a.x;
  io.y = a.y_scratch;
  io.gate = a.gate_scratch;
  io.rho = nullptr;          // rho goes to g.rho_scratch[0]
  io.step = nullptr;
  io.n_steps = 1;
  cudaError_t e;
  // pass 1: r1 = x - P (P^T x), rho
  if ((e = launch_project_residual(g, io, st)) != cudaSuccess) return e;
  k_ext_keep_rho<<<1, 32, 0, st>>>(g, a);
  // pass 2: r2 = r1 - P (P^T r1)
  if ((e = cudaMemcpyAsync(a.x_scratch, g.r, (size_t)g.d * sizeof(float), cudaMemcpyDeviceToDevice,
                           st)) != cudaSuccess)
    return e;
  io.x = a.x_scratch;
  if ((e = launch_project_residual(g, io, st)) != cudaSuccess) return e;
  k_ext_decide<<<1, kExtThreads, 0, st>>>(g, a);
  k_ext_store_vector<<<(g.d + 255) / 256, 256, 0, st>>>(g, a);
  // image column: y_scratch = W v through the gated-residual GEMV (one pass over W)
  if ((e = cudaMemsetAsync(a.y_scratch, 0, (size_t)g.O * sizeof(float), st)) != cudaSuccess) return e;
  if ((e = launch_gated_gemv(g, io, st)) != cudaSuccess) return e;
  k_ext_store_image<<<(g.O + 255) / 256, 256, 0, st>>>(g, a);
  return cudaGetLastError();
}

}  // namespace gsi
