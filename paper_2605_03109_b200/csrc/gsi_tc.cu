// Gated residual for MANY fired tokens as a dense contraction on the 5th-gen
// tensor cores (Eq. (3.2): y_t += W r_t for every gated token t of the batch).
//
// Swap-AB formulation: the accumulator tile is D[128 rows of W][N tokens], N the
// fired-token count padded to a multiple of 16 (16..64).  W is streamed exactly
// once per step; the contraction stays HBM-bound (<= 64 FLOP/B, far below the
// tensor ridge), the tensor pipe is only the means to stay on the HBM roofline
// once there are too many tokens for CUDA-core FMAs.
//
//   A (W tile, 128 x 64 bf16 per stage)   global -> shared by TMA in the 128-byte-swizzled
//   B (R tile,   N x 64 bf16 per stage)   K-major layout tcgen05 reads
//   D (128 lanes x N columns fp32)        tensor memory; tcgen05.mma, one issuing thread
//   epilogue                              tcgen05.ld -> registers -> partial-sum buffer
//
// Split-K over CTAs fills the machine for the narrow maps; partial sums are added
// to y in a fixed order by a second small kernel, so results are reproducible.
// Every wait is bounded; a timeout sets the status word, frees the tensor memory
// and returns.
#include "gsi_umma.cuh"

namespace gsi {

namespace {

using namespace umma;

constexpr int kStages = 4;   // 4 x 24 KB, two blocks per SM (8 stages x 1 block and 3 x 3 measured slower)
constexpr int kMaxN = 64;
constexpr int kTmemCols = 64;
constexpr int kSpeculateTokens = 16;   // tokens per call from which W tiles are requested before the gate is known
using TcCfg = Cfg<kStages, kMaxN>;
constexpr int kThreadsTc = kThreads;
constexpr int kTcSmem = TcCfg::kSmem;

// r (fp32, all tokens) -> Rb (bf16, fired tokens compacted, zero rows up to 64)
__global__ void __launch_bounds__(256) k_pack_fired_bf16(GroupParams g, int min_fired) {
  const int n = *g.n_fired;
  if (n < min_fired) return;
  const int row = blockIdx.y;  // 0..63
  const int tok = row < n ? g.fired[row] : -1;
  for (int i = blockIdx.x * 256 + threadIdx.x; i < g.d; i += gridDim.x * 256) {
    const float v = tok >= 0 ? g.r[(size_t)tok * g.d + i] : 0.f;
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    g.rb[(size_t)row * g.d + i] = *reinterpret_cast<const uint16_t*>(&h);
  }
}

// mapped == 0: B rows are the fired tokens compacted (N = fired count rounded up to 16).
// mapped == 1: B rows are all n_tokens tokens of the call (row = token); only the columns
//              of fired tokens are written out.
__global__ void __launch_bounds__(kThreadsTc, 2)
k_residual_gemm_tc(GroupParams g, const __grid_constant__ TmaMaps tm, IoRef io, int min_fired, int splits,
                   int mapped, int n_tokens) {
  pdl_launch_dependents();
  // With many tokens per call some token is gated nearly always: the W tiles are then
  // requested before the fired list of the kernel before is known (mapped operand rows only:
  // their number does not depend on the list), and the block backs out if nobody fired.
  const bool speculate = mapped && n_tokens >= kSpeculateTokens;
  int n_fired = 0;
  if (!speculate) {
    pdl_wait();   // the fired list comes from the kernel before
    n_fired = *g.n_fired;
    if (n_fired < min_fired) return;          // nothing gated, or the CUDA-core GEMV takes the few
  }
  const int n_cols = mapped ? n_tokens : n_fired;
  const int N = (n_cols + 15) & ~15;          // 16..64

  extern __shared__ unsigned char smem_raw[];
  __shared__ unsigned long long s_mask;       // columns to write out
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x / splits, split = blockIdx.x % splits;
  const int row0 = tile * kTM;                 // first row of the concatenated maps
  int j = 0;
  while (j + 1 < g.n_maps && row0 >= g.off[j + 1]) ++j;   // a tile never straddles two maps
  const int nkb = g.d / kTK;
  const int kb0 = (int)((long long)nkb * split / splits), kb1 = (int)((long long)nkb * (split + 1) / splits);
  const int nloc = kb1 - kb0;

  uint32_t tmem;
  bool skipped = false;
  const bool ok = tile_mma<kStages, kMaxN, kTmemCols>(smem_raw, &tm.w[j], row0 - g.off[j], &tm.rb, 0, N,
                                                      kb0, nloc, &tmem, speculate ? g.n_fired : nullptr,
                                                      min_fired, &skipped);
  if (!skipped) {   // past the wait on the kernel before: the fired list is there
    if (threadIdx.x == 0) {
      n_fired = *g.n_fired;
      unsigned long long m = 0ull;
      if (mapped) {
        for (int n = 0; n < n_fired; ++n) m |= 1ull << g.fired[n];
      } else {
        m = n_fired >= 64 ? ~0ull : ((1ull << n_fired) - 1ull);
      }
      s_mask = m;
    }
    __syncthreads();
  }
  if (skipped) {
    // nothing to write
  } else if (!ok) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)GSI_ERR_TIMEOUT);
  } else if (nloc > 0) {
    // warp w owns tensor-memory lanes 32w..32w+31 = rows row0+32w+lane; 16 columns per load
    // One split: the tile's rows belong to this block alone, and y holds the image product of
    // the kernels before: the sums are added to y here (no partial sums, no second kernel).
    const unsigned long long mask = s_mask;
    const int row = row0 + warp * 32 + lane;
    float* yp = g.ypart + ((size_t)split * kMaxN) * g.O + row;
    for (int c0 = 0; c0 < N; c0 += 16) {
      if (((mask >> c0) & 0xFFFFull) == 0ull) continue;
      uint32_t v[16];
      tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
      tmem_ld_wait();
      if (splits == 1) {
        // (an addition at the L2 without a round trip; one writer per element, so the result
        // does not depend on any order)
#pragma unroll
        for (int c = 0; c < 16; ++c)
          if ((mask >> (c0 + c)) & 1ull) {
            const int tok = mapped ? c0 + c : g.fired[c0 + c];
            asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(io.y + (size_t)tok * g.O + row),
                         "f"(__uint_as_float(v[c]))
                         : "memory");
          }
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c)
          if ((mask >> (c0 + c)) & 1ull) yp[(size_t)(c0 + c) * g.O] = __uint_as_float(v[c]);
      }
    }
  }
  tile_release<kTmemCols>(tmem);
}

// y[fired[n]][row] += sum over splits (fixed order); the partial sums of fired token n
// are column n (compacted) or column fired[n] (mapped)
__global__ void __launch_bounds__(256) k_add_partials(GroupParams g, IoRef io, int min_fired, int splits,
                                                      int mapped) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = *g.n_fired;
  if (n < min_fired) return;
  const int t = blockIdx.y;
  if (t >= n) return;
  const int tok = g.fired[t];
  const int col = mapped ? tok : t;
  for (int row = blockIdx.x * 256 + threadIdx.x; row < g.O; row += gridDim.x * 256) {
    float s = 0.f;
    for (int sp = 0; sp < splits; ++sp) s += g.ypart[((size_t)sp * kMaxN + col) * g.O + row];
    io.y[(size_t)tok * g.O + row] += s;
  }
}

// ---- dense baseline for batched calls: y = W bf16(x) on the same tile routine -----------
// The activations are rounded to bf16 as an ordinary bf16 GEMM would take them (one operand
// row per token), which makes this the strongest dense comparator the tile routine offers:
// the stage size and occupancy of the gated-residual GEMM, no pack by a fired list.
__global__ void __launch_bounds__(256) k_pack_x_bf16(GroupParams g, IoRef io, int n_tokens) {
  // first kernel of the chain: wait first (rb may still be read by the previous call's GEMM,
  // and the GEMM after this kernel requests weight tiles before its own wait)
  pdl_wait();
  pdl_launch_dependents();
  const int row = blockIdx.y;   // operand row = token; rows up to the next multiple of 16 are zero
  const float* x = io.x + (long long)io_slot(io) * io.x_step_stride + (size_t)row * g.d;
  for (int i = blockIdx.x * 256 + threadIdx.x; i < g.d; i += gridDim.x * 256) {
    const float v = row < n_tokens ? __ldg(x + i) : 0.f;
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    g.rb[(size_t)row * g.d + i] = *reinterpret_cast<const uint16_t*>(&h);
  }
}

__global__ void __launch_bounds__(kThreadsTc, 2)
k_dense_gemm_tc(GroupParams g, const __grid_constant__ TmaMaps tm, IoRef io, int splits, int n_tokens) {
  extern __shared__ unsigned char smem_raw[];
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x / splits, split = blockIdx.x % splits;
  const int row0 = tile * kTM;
  int j = 0;
  while (j + 1 < g.n_maps && row0 >= g.off[j + 1]) ++j;
  const int nkb = g.d / kTK;
  const int kb0 = (int)((long long)nkb * split / splits), kb1 = (int)((long long)nkb * (split + 1) / splits);
  const int N = (n_tokens + 15) & ~15;
  uint32_t tmem;
  const bool ok = tile_mma<kStages, kMaxN, kTmemCols>(smem_raw, &tm.w[j], row0 - g.off[j], &tm.rb, 0, N,
                                                      kb0, kb1 - kb0, &tmem);
  if (!ok) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)GSI_ERR_TIMEOUT);
  } else {
    // (one split: straight to y, and this kernel reports every token as gated)
    const int row = row0 + warp * 32 + lane;
    float* yp = g.ypart + ((size_t)split * kMaxN) * g.O + row;
    if (splits == 1 && blockIdx.x == 0 && threadIdx.x < n_tokens)
      io.gate[(long long)io_slot(io) * io.log_step_stride + threadIdx.x] = 1;
    for (int c0 = 0; c0 < N; c0 += 16) {
      uint32_t v[16];
      tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
      tmem_ld_wait();
#pragma unroll
      for (int c = 0; c < 16; ++c)
        if (c0 + c < n_tokens) {
          if (splits == 1)
            io.y[(size_t)(c0 + c) * g.O + row] = __uint_as_float(v[c]);
          else
            yp[(size_t)(c0 + c) * g.O] = __uint_as_float(v[c]);
        }
    }
  }
  tile_release<kTmemCols>(tmem);
}

// y[t][row] = sum over splits (fixed order); the dense baseline reports every token as gated
__global__ void __launch_bounds__(256) k_sum_partials(GroupParams g, IoRef io, int splits, int n_tokens) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.y;
  if (blockIdx.x == 0 && threadIdx.x == 0)
    io.gate[(long long)io_slot(io) * io.log_step_stride + t] = 1;
  for (int row = blockIdx.x * 256 + threadIdx.x; row < g.O; row += gridDim.x * 256) {
    float s = 0.f;
    for (int sp = 0; sp < splits; ++sp) s += g.ypart[((size_t)sp * kMaxN + t) * g.O + row];
    io.y[(size_t)t * g.O + row] = s;
  }
}

}  // namespace

cudaError_t launch_dense_gemm_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io, int n_tokens,
                                 cudaStream_t st, int* n_launches) {
  cudaError_t e = cudaFuncSetAttribute(k_dense_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kTcSmem);
  if (e != cudaSuccess) return e;
  const int splits = tc_splits(g.O, g.d);
  const int rows = (n_tokens + 15) & ~15;
  k_pack_x_bf16<<<dim3((g.d + 2047) / 2048, rows), 256, 0, st>>>(g, io, n_tokens);
  if ((e = launch_pdl(k_dense_gemm_tc, dim3((g.O / kTM) * splits), dim3(kThreadsTc), kTcSmem, st, g, tm, io,
                      splits, n_tokens)) != cudaSuccess)
    return e;
  if (splits > 1 &&
      (e = launch_pdl(k_sum_partials, dim3((g.O + 1023) / 1024, n_tokens), dim3(256), 0, st, g, io, splits,
                      n_tokens)) != cudaSuccess)
    return e;
  if (n_launches) *n_launches += splits > 1 ? 3 : 2;
  return cudaGetLastError();
}

int tc_splits(int O, int d) {
  const int tiles = O / kTM, nkb = d / kTK;
  if (tiles >= 148) return 1;   // a tile per CTA already fills the SMs: long pipelines, no partial sums to add
  int s = (2 * 148 + tiles - 1) / tiles;
  if (s > 8) s = 8;
  if (s > nkb / 4) s = nkb / 4;
  if (s < 1) s = 1;
  return s;
}

bool tc_eligible(const GroupParams& g) {
  if (g.d % kTK) return false;
  for (int j = 0; j < g.n_maps; ++j)
    if (g.d_out[j] % kTM) return false;
  return true;
}

cudaError_t launch_residual_gemm_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io,
                                    int min_fired, bool mapped, int n_tokens, cudaStream_t st,
                                    int* n_launches) {
  cudaError_t e = cudaFuncSetAttribute(k_residual_gemm_tc,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
  if (e != cudaSuccess) return e;
  const int splits = tc_splits(g.O, g.d);
  if (!mapped) k_pack_fired_bf16<<<dim3((g.d + 2047) / 2048, kMaxN), 256, 0, st>>>(g, min_fired);
  if (mapped) {
    // straight after the residual kernel: both may start while their predecessor drains
    if ((e = launch_pdl(k_residual_gemm_tc, dim3((g.O / kTM) * splits), dim3(kThreadsTc), kTcSmem, st, g,
                        tm, io, min_fired, splits, 1, n_tokens)) != cudaSuccess)
      return e;
    if (splits > 1 &&
        (e = launch_pdl(k_add_partials, dim3((g.O + 1023) / 1024, g.B), dim3(256), 0, st, g, io,
                        min_fired, splits, 1)) != cudaSuccess)
      return e;
  } else {
    k_residual_gemm_tc<<<(g.O / kTM) * splits, kThreadsTc, kTcSmem, st>>>(g, tm, io, min_fired, splits, 0,
                                                                          n_tokens);
    if (splits > 1) k_add_partials<<<dim3((g.O + 1023) / 1024, g.B), 256, 0, st>>>(g, io, min_fired, splits, 0);
  }
  if (n_launches) *n_launches += (mapped ? 1 : 2) + (splits > 1 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace gsi
