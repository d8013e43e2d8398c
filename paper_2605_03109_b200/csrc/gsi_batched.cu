// Batched front end of the gated subspace layer on the 5th-gen tensor cores:
// Algorithm 1 lines 1-5 for a batch of tokens as three skinny contractions,
//
//   c  = P^T x      A = P^T tile [128 of k][d],   B = terms of x [3n][d],  split over d
//   Pc (-> r, gate) A = P tile   [128 of d][k],   B = terms of c [3n][k]
//   y  = W_P c      A = W_P tile [128 of O][k],   B = terms of c [3n][k]
//
// The basis and the images are bf16 already; the fp32 activations and coefficients
// enter as THREE bf16 terms each (v = hi + mid + lo, 24 significant bits), stored as
// rows 3t, 3t+1, 3t+2 of the B operand, so every product is exact and the sums are
// fp32 in tensor memory: the same arithmetic as the CUDA-core kernels up to the order
// of the additions.  The epilogues add the three columns of a token and apply the rest
// of the line: the split-K partial of c; r = x - Pc with the partial sums of ||r||^2
// and ||x||^2 followed by the gate decision (Eq. (3.3)) in the last block; y.
#include "gsi_umma.cuh"

namespace gsi {

namespace {

using namespace umma;

constexpr int kStages3 = 4;
constexpr int kMaxN3 = 192;          // 3 terms x 64 tokens
constexpr int kTmemCols3 = 256;      // power of two >= kMaxN3
using Cfg3 = Cfg<kStages3, kMaxN3>;
constexpr int kSmem3 = Cfg3::kSmem;  // 4 x (16 + 24) KB + slack
// residual / image: K = k is short (four 64-wide blocks at k = 256).  Up to 32 tokens the B
// operand is small enough for four stages with two blocks per SM, so every weight box of a
// tile is requested before the wait on the previous kernel; beyond, two stages.
constexpr int kStagesRI = 2, kStagesRIs = 4;
constexpr int kMaxN3s = 96, kTmemCols3s = 128;   // 3 terms x 32 tokens
constexpr int kSmemRI = Cfg<kStagesRI, kMaxN3>::kSmem;
constexpr int kSmemRIs = Cfg<kStagesRIs, kMaxN3s>::kSmem;

__device__ __forceinline__ uint16_t bf16_bits(float v) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  return *reinterpret_cast<const uint16_t*>(&h);
}
__device__ __forceinline__ float bf16_val(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// v = hi + mid + lo exactly for every finite fp32 v whose low term is not subnormal.
__device__ __forceinline__ void split3(float v, uint16_t& hi, uint16_t& mid, uint16_t& lo) {
  hi = bf16_bits(v);
  const float r1 = v - bf16_val(hi);
  mid = bf16_bits(r1);
  const float r2 = r1 - bf16_val(mid);
  lo = bf16_bits(r2);
}

__device__ __forceinline__ int rows3(int n_tokens) { return term_rows(n_tokens); }

// src [n_tokens][len] fp32 -> dst [rows3][len] bf16 terms; rows past 3 n_tokens are zero.
// One block row (blockIdx.y) per token slot, 8 elements per thread.
__device__ __forceinline__ void store_terms(const float (&v)[8], bool live, uint16_t* dst, int slot,
                                            int n_rows, size_t len, size_t at) {
  uint32_t w[3][4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    uint16_t a[3], b[3];
    if (live) {
      split3(v[2 * e], a[0], a[1], a[2]);
      split3(v[2 * e + 1], b[0], b[1], b[2]);
    } else {
      a[0] = a[1] = a[2] = b[0] = b[1] = b[2] = 0;
    }
#pragma unroll
    for (int c = 0; c < 3; ++c) w[c][e] = (uint32_t)a[c] | ((uint32_t)b[c] << 16);
  }
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    const int row = 3 * slot + c;
    if (row < n_rows)
      *reinterpret_cast<uint4*>(dst + (size_t)row * len + at) = make_uint4(w[c][0], w[c][1], w[c][2], w[c][3]);
  }
}

__global__ void __launch_bounds__(256) k_split3_x(GroupParams g, IoRef io, int n_tokens) {
  // first kernel of the chain: wait first, so that nothing of the chain (its successors
  // request weight tiles before their own waits) runs beside an earlier call's kernels
  pdl_wait();   // xb may still be read by the previous call's projection
  pdl_launch_dependents();
  const int slot = blockIdx.y, n_rows = rows3(n_tokens);
  const bool live = slot < n_tokens;
  const float* x = io.x + (long long)io_slot(io) * io.x_step_stride + (size_t)slot * g.d;
  for (int i8 = blockIdx.x * 256 + threadIdx.x; i8 < g.d / 8; i8 += gridDim.x * 256) {
    float v[8] = {};
    if (live) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(x) + 2 * i8);
      const float4 b = __ldg(reinterpret_cast<const float4*>(x) + 2 * i8 + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
      v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
    store_terms(v, live, g.xb, slot, n_rows, (size_t)g.d, (size_t)i8 * 8);
  }
}

// c partials: cpart3[split][t][128*tile + lane row] over this split's share of d.
__global__ void __launch_bounds__(kThreads, 1)
k_proj_tc(GroupParams g, const __grid_constant__ TmaMaps tm, int n_tokens) {
  extern __shared__ unsigned char smem_raw[];
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int splits = g.proj_splits;
  const int tile = blockIdx.x / splits, split = blockIdx.x % splits;
  const int nkb = g.d / kTK;
  const int kb0 = (int)((long long)nkb * split / splits), kb1 = (int)((long long)nkb * (split + 1) / splits);
  uint32_t tmem;
  const bool ok = tile_mma<kStages3, kMaxN3, kTmemCols3>(smem_raw, &tm.pt, tile * kTM, &tm.xb, 0,
                                                         rows3(n_tokens), kb0, kb1 - kb0, &tmem);
  if (!ok) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)GSI_ERR_TIMEOUT);
  } else {
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    float* out = g.cpart3 + (size_t)split * g.B * g.k + tile * kTM + warp * 32 + lane;
    for (int q = 0; 16 * q < n_tokens; ++q) {
      float s[16];
      sum3_tokens16(tl, q, s);
#pragma unroll
      for (int tt = 0; tt < 16; ++tt)
        if (16 * q + tt < n_tokens) out[(size_t)(16 * q + tt) * g.k] = s[tt];
    }
  }
  tile_release<kTmemCols3>(tmem);
}

// c = sum of the split-K partials in split order; also its three bf16 terms.
// One block per token slot, one coefficient per thread and pass.
__global__ void __launch_bounds__(256) k_reduce_split3_c(GroupParams g, int n_tokens) {
  const int slot = blockIdx.x, n_rows = rows3(n_tokens);
  const bool live = slot < n_tokens;
  pdl_launch_dependents();
  pdl_wait();
  for (int j = threadIdx.x; j < g.k; j += 256) {
    float v = 0.f;
    if (live) {
      const float* p = g.cpart3 + (size_t)slot * g.k + j;
      const size_t stride = (size_t)g.B * g.k;
      int s = 0;
      for (; s + 32 <= g.proj_splits; s += 32) {   // thirty-two partials in flight, summed in order
        float u[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) u[i] = p[(size_t)(s + i) * stride];
#pragma unroll
        for (int i = 0; i < 32; ++i) v += u[i];
      }
      for (; s + 8 <= g.proj_splits; s += 8) {
        float u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) u[i] = p[(size_t)(s + i) * stride];
#pragma unroll
        for (int i = 0; i < 8; ++i) v += u[i];
      }
      for (; s < g.proj_splits; ++s) v += p[(size_t)s * stride];
      g.c[(size_t)slot * g.k + j] = v;
    }
    uint16_t term[3] = {0, 0, 0};
    if (live) split3(v, term[0], term[1], term[2]);
#pragma unroll
    for (int c = 0; c < 3; ++c)
      if (3 * slot + c < n_rows) g.cb[(size_t)(3 * slot + c) * g.k + j] = term[c];
  }
}

// One launch for Algorithm 1 lines 2-5.  Every block contracts one 128-row tile against
// the c terms of a range of 16-token groups (operand rows 48 q_lo .. 48 q_hi - 1):
//   blocks [0, n_resid)   tile of P, one of rs token ranges (rs > 1 spreads the narrow
//                         inputs, d = 4096: 32 tiles, over the machine):
//                         r = x - P c -> bf16 rows of rb, the partial norms of the tile,
//                         and in the block that finishes last the gate
//   blocks [n_resid, ..)  tile of W_P, all tokens: y = W_P c
template <int kStagesT, int kMaxRows, int kTmemColsT>
__global__ void __launch_bounds__(kThreads, 2)
k_resid_image_tc(GroupParams g, const __grid_constant__ TmaMaps tm, IoRef io, int n_tokens, int rs) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ float s_norm[kThreads / 32][GSI_MAX_TOKENS][2];
  __shared__ int s_last;
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = (n_tokens + 15) / 16;
  const int n_resid = (g.d / kTM) * rs;
  const bool image = (int)blockIdx.x >= n_resid;
  const int tile = image ? (int)blockIdx.x - n_resid : (int)blockIdx.x / rs;
  const int part = image ? 0 : (int)blockIdx.x % rs;
  const int per = image ? nq : (nq + rs - 1) / rs;
  const int q_lo = min(part * per, nq), q_hi = min(q_lo + per, nq);
  const int row = tile * kTM + warp * 32 + lane;
  const int slot = io_slot(io);
  const float* x = io.x + (long long)slot * io.x_step_stride + row;

  float xv[16];
  if (!image && q_lo < q_hi) {
#pragma unroll
    for (int tt = 0; tt < 16; ++tt)
      xv[tt] = (16 * q_lo + tt < n_tokens) ? __ldg(x + (size_t)(16 * q_lo + tt) * g.d) : 0.f;
  }
  uint32_t tmem = 0;
  bool ok = true;
  if (q_lo < q_hi) {   // block-uniform
    const int n_rows = min(48 * (q_hi - q_lo), rows3(n_tokens) - 48 * q_lo);
    ok = tile_mma<kStagesT, kMaxRows, kTmemColsT>(smem_raw, image ? &tm.wp : &tm.p, tile * kTM, &tm.cb,
                                                48 * q_lo, n_rows, 0, g.k / kTK, &tmem);
    if (!ok && threadIdx.x == 0) atomicExch(g.status, (int)GSI_ERR_TIMEOUT);
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    for (int q = q_lo; q < q_hi && ok; ++q) {
      float s[16];
      sum3_tokens16(tl, q - q_lo, s);
      if (image) {
#pragma unroll
        for (int tt = 0; tt < 16; ++tt)
          if (16 * q + tt < n_tokens) io.y[(size_t)(16 * q + tt) * g.O + row] = s[tt];
        continue;
      }
      float xn[16];   // the next group's x, in flight while this group is reduced
#pragma unroll
      for (int tt = 0; tt < 16; ++tt)
        xn[tt] = (q + 1 < q_hi && 16 * (q + 1) + tt < n_tokens) ? __ldg(x + (size_t)(16 * (q + 1) + tt) * g.d)
                                                                 : 0.f;
#pragma unroll
      for (int tt = 0; tt < 16; ++tt) {
        const int t = 16 * q + tt;
        const float rv = xv[tt] - s[tt];
        if (t < n_tokens) g.rb[(size_t)t * g.d + row] = bf16_bits(rv);
        const float a = warp_sum(rv * rv), b = warp_sum(xv[tt] * xv[tt]);
        if (lane == 0 && t < n_tokens) {
          s_norm[warp][t][0] = a;
          s_norm[warp][t][1] = b;
        }
        xv[tt] = xn[tt];
      }
    }
    tile_release<kTmemColsT>(tmem);
  }
  if (image) return;
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * (q_hi - q_lo); i += kThreads) {
    const int t = 16 * q_lo + (i >> 1), w = i & 1;
    if (t < n_tokens) {
      float sum = 0.f;
#pragma unroll
      for (int wp = 0; wp < kThreads / 32; ++wp) sum += ok ? s_norm[wp][t][w] : 0.f;
      g.normpart3[((size_t)tile * g.B + t) * 2 + w] = sum;
    }
  }
  decide_gate_last_block(g, io, slot, n_tokens, g.normpart3, g.d / kTM, (unsigned)n_resid, &s_last);
}

// PT[j][i] = P[i][j], 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) k_transpose_bf16(const uint16_t* __restrict__ P, int d, int k,
                                                        uint16_t* __restrict__ PT) {
  __shared__ uint16_t tile[32][33];
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8)
    if (i0 + r < d && j0 + tx < k) tile[r][tx] = P[(size_t)(i0 + r) * k + j0 + tx];
  __syncthreads();
  for (int r = ty; r < 32; r += 8)
    if (j0 + r < k && i0 + tx < d) PT[(size_t)(j0 + r) * d + i0 + tx] = tile[tx][r];
}

}  // namespace

int front_rows(int max_tokens) { return (3 * max_tokens + 15) & ~15; }

int front_proj_splits(int d, int k) {
  const int tiles = k / kTM, nkb = d / kTK;
  int s = 148 / tiles;
  if (s > nkb / 2) s = nkb / 2;
  if (s > 32) s = 32;   // more partials cost the reduction more than they save the projection (measured)
  if (s < 1) s = 1;
  return s;
}

cudaError_t launch_transpose_bf16(const void* P, int d, int k, void* PT, cudaStream_t st) {
  k_transpose_bf16<<<dim3((k + 31) / 32, (d + 31) / 32), 256, 0, st>>>(
      static_cast<const uint16_t*>(P), d, k, static_cast<uint16_t*>(PT));
  return cudaGetLastError();
}

cudaError_t launch_split3_x(const GroupParams& g, const IoRef& io, int n_tokens, cudaStream_t st) {
  const int slots = (front_rows(n_tokens) + 2) / 3;
  k_split3_x<<<dim3((g.d / 8 + 255) / 256, slots), 256, 0, st>>>(g, io, n_tokens);
  return cudaGetLastError();
}

cudaError_t launch_front_tc(const GroupParams& g, const TmaMaps& tm, const IoRef& io, int n_tokens,
                            cudaStream_t st, int* n_launches) {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_proj_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem3)) != cudaSuccess ||
      (e = cudaFuncSetAttribute(k_resid_image_tc<kStagesRI, kMaxN3, kTmemCols3>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemRI)) != cudaSuccess ||
      (e = cudaFuncSetAttribute(k_resid_image_tc<kStagesRIs, kMaxN3s, kTmemCols3s>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemRIs)) != cudaSuccess)
    return e;
  const bool small = term_rows(n_tokens) <= kMaxN3s;
  const int slots = (front_rows(n_tokens) + 2) / 3;   // token slots covering every operand row
  const int nq = (n_tokens + 15) / 16, tiles = g.d / kTM;
  int rs = tiles <= 37 ? 4 : tiles <= 148 ? 2 : 1;   // token ranges per residual tile (measured: 4 for all is slower)
  if (rs > nq) rs = nq;
  // the x the residual blocks read before their wait is an input of the call, complete before
  // k_split3_x was launched
  if ((e = launch_pdl(k_split3_x, dim3((g.d / 8 + 255) / 256, slots), dim3(256), 0, st, g, io, n_tokens)) !=
          cudaSuccess ||
      (e = launch_pdl(k_proj_tc, dim3((g.k / kTM) * g.proj_splits), dim3(kThreads), kSmem3, st, g, tm,
                      n_tokens)) != cudaSuccess ||
      (e = launch_pdl(k_reduce_split3_c, dim3(slots), dim3(256), 0, st, g, n_tokens)) != cudaSuccess ||
      (e = small ? launch_pdl(k_resid_image_tc<kStagesRIs, kMaxN3s, kTmemCols3s>,
                              dim3((g.d / kTM) * rs + g.O / kTM), dim3(kThreads), kSmemRIs, st, g, tm, io,
                              n_tokens, rs)
                 : launch_pdl(k_resid_image_tc<kStagesRI, kMaxN3, kTmemCols3>,
                              dim3((g.d / kTM) * rs + g.O / kTM), dim3(kThreads), kSmemRI, st, g, tm, io,
                              n_tokens, rs)) != cudaSuccess)
    return e;
  if (n_launches) *n_launches += 4;
  return cudaGetLastError();
}

}  // namespace gsi
