// Shared device helpers and internal declarations of the gated subspace layer.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "gsi.h"

namespace gsi {

constexpr int kWarp = 32;
constexpr int kTokChunk = 4;  // tokens held in registers at once by the generic kernels

// Where a group's activations and logs live for the current decode step.  A
// plain gsi_forward call has step == nullptr (offset 0).
struct IoRef {
  const float* x;       // [n_steps][B][d] (or [B][d])
  float* y;             // [B][O]
  unsigned char* gate;  // [n_steps][log_groups][B] (or [B])
  float* rho;           // same shape as gate, or nullptr
  const int* step;      // device step counter or nullptr
  int n_steps;
  long long x_step_stride;    // elements between steps of x
  long long log_step_stride;  // elements between steps of gate / rho
};

__device__ __forceinline__ int io_slot(const IoRef& io) {
  return io.step ? (*io.step % io.n_steps) : 0;
}

// 8 consecutive basis / image entries as fp32.
__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float (&f)[8]) {
  f[0] = __uint_as_float(v.x << 16);
  f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16);
  f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16);
  f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16);
  f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

// Element index `idx8` counts groups of 8 elements from `base`.
template <bool kF32>
__device__ __forceinline__ void load8(const void* base, size_t idx8, float (&f)[8]) {
  if constexpr (kF32) {
    const float4* p = reinterpret_cast<const float4*>(base) + idx8 * 2;
    float4 a = __ldg(p), b = __ldg(p + 1);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
    f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
  } else {
    uint4 v = __ldg(reinterpret_cast<const uint4*>(base) + idx8);
    unpack_bf16x8(v, f);
  }
}

// One-shot weight stream: do not keep it in L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Programmatic dependent launch.  A kernel calls pdl_launch_dependents() first, so the next
// kernel of the stream (if it was launched with launch_pdl) may be scheduled and run its
// set-up while this one finishes, and pdl_wait() before it touches anything an earlier kernel
// of the stream wrote or still reads; the wait returns once every earlier kernel has completed
// and flushed.  Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- generic path (any supported shape, any batch <= GSI_MAX_TOKENS) --------
struct GroupParams {
  int d, k, O, B;            // O = sum of d_out
  int p_f32;                 // basis stored as fp32
  float eps;
  unsigned flags;
  const void* P;             // [d][k]
  const uint16_t* WP;        // [O][k] bf16 (concatenated images)
  int n_maps;
  const uint16_t* W[GSI_MAX_MAPS];  // [d_out_j][d] bf16
  int d_out[GSI_MAX_MAPS];
  int off[GSI_MAX_MAPS + 1];
  // scratch
  float* c;         // [B][k]
  float* cpart;     // [n_slabs][B][k]
  float* r;         // [B][d]
  float* normpart;  // [n_slabs][B][2]
  int* fired;       // [B] token indices, ascending
  int* n_fired;     // [1]
  unsigned* counter;  // [1] arrival counter of the residual kernel
  float* rho_scratch; // [B]
  int* status;      // [1]
  int n_slabs, slab_rows;
  // tensor-core gated residual (batched): used when at least tc_min_fired tokens fired
  int tc_min_fired;   // 0 = disabled
  uint16_t* rb;       // [65][d] bf16 residuals: fired tokens compacted, or (batched front end)
                      // row t = token t; row 64 stays zero
  float* ypart;       // [splits][64][O] split-K partial sums
  // tensor-core projection / residual / image (batched): used for calls with at least
  // front_min_tokens tokens.  fp32 operands enter as three bf16 terms (row 3t+c of the
  // B operand is term c of token t), so products are exact and sums are fp32.
  int front_min_tokens;   // 0 = disabled
  int proj_splits;        // split-K CTAs per 128 columns of the projection
  const uint16_t* PT;     // [k][d] bf16: the basis transposed (K-major for c = P^T x)
  uint16_t* xb;           // [3B rounded up to 16][d] bf16 terms of x
  uint16_t* cb;           // [3B rounded up to 16][k] bf16 terms of c
  float* cpart3;          // [proj_splits][B][k] split-K partial sums of c
  float* normpart3;       // [d/128][B][2] per-tile partial sums of ||r||^2, ||x||^2
};

// The block that arrives last (of n_blocks) sums the per-part norm partials in part
// order in double precision, writes gate / rho (Eq. (3.3)) and the ascending list of
// fired tokens, and rearms the arrival counter.  Every thread of every block calls it
// after its partials are written; s_last is a shared-memory word.
__device__ __forceinline__ void decide_gate_last_block(const GroupParams& g, const IoRef& io,
                                                       int slot, int n_tokens,
                                                       const float* normpart, int n_parts,
                                                       unsigned n_blocks, int* s_last) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(g.counter, 1u);
    *s_last = (prev == n_blocks - 1);
  }
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  __shared__ unsigned char s_gate[GSI_MAX_TOKENS];   // the decisions, for the list of gated tokens
  unsigned char* gate = io.gate + (long long)slot * io.log_step_stride;
  float* rho = io.rho ? io.rho + (long long)slot * io.log_step_stride : g.rho_scratch;
  // L adjacent lanes share a token: each sums a contiguous range of parts in order (loads
  // issued thirty-two parts at a time), then the L sums are combined by a butterfly, so the
  // result depends on n_tokens and the block size only through L and is reproducible.
  int L = 1;
  while (2 * L <= 32 && 2 * L * n_tokens <= (int)blockDim.x) L *= 2;
  const int per_pass = blockDim.x / L;
  for (int t0 = 0; t0 < n_tokens; t0 += per_pass) {   // block-uniform trip count
    const int t = t0 + (int)threadIdx.x / L, l = (int)threadIdx.x % L;
    const bool live = t < n_tokens;
    const int p0 = (int)((long long)n_parts * l / L), p1 = (int)((long long)n_parts * (l + 1) / L);
    double sr = 0.0, sx = 0.0;
    if (live) {
      const float2* np = reinterpret_cast<const float2*>(normpart) + t;
      for (int p = p0; p < p1; p += 32) {
        float2 v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u)
          v[u] = (p + u < p1) ? __ldcg(np + (size_t)(p + u) * g.B) : make_float2(0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          sr += (double)v[u].x;
          sx += (double)v[u].y;
        }
      }
    }
    for (int o = 1; o < L; o <<= 1) {
      sr += __shfl_xor_sync(0xffffffffu, sr, o);
      sx += __shfl_xor_sync(0xffffffffu, sx, o);
    }
    if (live && l == 0) {
      const double nr = sqrt(sr), nx = sqrt(sx);
      const bool fast = nr < (double)g.eps * nx;  // false for NaN and for x = 0
      gate[t] = fast ? 0 : 1;
      s_gate[t] = fast ? 0 : 1;
      rho[t] = (float)(nr / nx);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0;
    if (!(g.flags & GSI_FLAG_STATIC_PROJECTION)) {
      for (int t = 0; t < n_tokens; ++t)
        if (s_gate[t]) g.fired[n++] = t;
    }
    *g.n_fired = n;
    *g.counter = 0u;
  }
}

// Launch that lets the kernel start before its predecessor in the stream has finished
// (the kernel must call pdl_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

struct TmaMaps;   // tensor maps of the layer's matrices (null when no tensor-core path is on)

// A second stream for the gated-residual contraction of batched calls: the contraction of a
// group is ordered behind that group's residual/gate kernel by the event and may run beside the
// projection of the groups that follow (their inputs are staged before the step); the caller
// joins the stream back at the end of the step.
struct ResidualLane {
  cudaStream_t stream;
  cudaEvent_t ev;
  bool used;
};

cudaError_t launch_generic_forward(const GroupParams& g, const TmaMaps* tm, const IoRef& io,
                                   int n_tokens, cudaStream_t stream, int* n_launches,
                                   ResidualLane* lane = nullptr);
cudaError_t launch_advance_step(int* step, cudaStream_t stream);
// One token on CUDA cores: c, r = x - P c into g.r (x may be g.r itself), rho into
// g.rho_scratch[0] (or io.rho), gate byte, fired list.  No image product.
cudaError_t launch_project_residual(const GroupParams& g, const IoRef& io, cudaStream_t stream);
// io.y[0][:] += W g.r for the token in the fired list (nothing if the list is empty).
cudaError_t launch_gated_gemv(const GroupParams& g, const IoRef& io, cudaStream_t stream);
// Online basis extension by one vector (see gsi_extend_basis).
struct ExtendArgs {
  const float* x;        // [d] the token
  float tau;
  int* k_active;         // device, in/out
  int* appended_out;     // device or null
  float* rho_out;        // device or null
  float* y_scratch;      // [O] device
  unsigned char* gate_scratch;  // [1] device
  int* ctrl;             // [4] device: appended, column, spare, spare
  float* inv_norm;       // [2] device: 1/||r2||, rho of the token
  float* x_scratch;      // [d] device: r1, the input of the second pass
  float* pmax;           // [1] device: max |P| of the handle (bf16 basis) or null
  uint16_t* PT;          // [k][d] transposed copy to keep in step, or null
};
cudaError_t launch_extend_basis(const GroupParams& g, const ExtendArgs& a, cudaStream_t stream);
// mapped: rb holds every token's residual (row = token) and the fired list selects the
// operand rows; otherwise a pack kernel first compacts the fired tokens of g.r into rb.
cudaError_t launch_residual_gemm_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io,
                                    int min_fired, bool mapped, int n_tokens,
                                    cudaStream_t stream, int* n_launches);
int tc_splits(int O, int d);
bool tc_eligible(const GroupParams& g);
// Batched front end on the tensor cores: c, r, gate and y = W_P c for n_tokens tokens.
cudaError_t launch_front_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io,
                            int n_tokens, cudaStream_t stream, int* n_launches);
// Encodes the layer's tensor maps (front: also those of the batched front end).
// False when the driver's encoder is unavailable or rejects a shape.
bool build_tma_maps(const GroupParams& g, bool front, int max_tokens, TmaMaps* out);
// xb = the three bf16 terms of every token of x (operand rows 3t, 3t+1, 3t+2).
cudaError_t launch_split3_x(const GroupParams& g, const IoRef& io, int n_tokens, cudaStream_t stream);
// Dense baseline for batched calls on the tensor cores: y = W bf16(x).
cudaError_t launch_dense_gemm_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io,
                                 int n_tokens, cudaStream_t stream, int* n_launches);
cudaError_t launch_transpose_bf16(const void* P, int d, int k, void* PT, cudaStream_t stream);
int front_proj_splits(int d, int k);
int front_rows(int max_tokens);   // rows of the three-term operands
// Kernel launches one generic forward of n_tokens tokens makes.
int generic_launch_count(const GroupParams& g, int n_tokens);
cudaError_t launch_build_image(const void* W, const void* P, int o, int d, int k, bool p_f32,
                               void* WP, cudaStream_t stream);

}  // namespace gsi
