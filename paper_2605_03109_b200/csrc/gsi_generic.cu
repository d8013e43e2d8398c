// Generic kernels of the gated subspace layer: any supported shape, any batch
// up to GSI_MAX_TOKENS, one launch per stage.  They follow Algorithm 1 stage by
// stage; the persistent decode kernel covers the same stages for the common
// shapes without the launch boundaries.
//
//   k_project_partial   c partials = P_slab^T x_slab          (Algorithm 1, line 1)
//   k_reduce_c          c = sum of partials, fixed order
//   k_residual_gate     r = x - P c, ||r||, ||x||, gate       (lines 2-4, Eq. (3.3))
//   k_image_gemv        y = W_P c                             (line 5)
//   k_stream_gemv       y += W r for gated tokens             (Eq. (3.2)), or the
//                       dense baseline y = W x
#include "gsi_common.cuh"

namespace gsi {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;
constexpr int TB = kTokChunk;

// A row of k entries is split into KV = k/8 vectors of 8.  LPR lanes share a
// row (a power of two <= 32), RPP = 32/LPR rows are processed per warp pass and
// each lane owns VPL = ceil(KV/LPR) vectors of every row it touches.
struct RowLayout {
  int KV, LPR, RPP, VPL;
};

__host__ __device__ inline RowLayout make_layout(int k) {
  RowLayout L;
  L.KV = k / 8;
  int lpr = 1;
  while (lpr < L.KV && lpr < 32) lpr <<= 1;
  L.LPR = lpr;
  L.RPP = 32 / lpr;
  L.VPL = (L.KV + lpr - 1) / lpr;
  return L;
}

template <int VPL, bool PF32>
__global__ void __launch_bounds__(kThreads)
k_project_partial(GroupParams g, IoRef io, int n_tokens) {
  extern __shared__ float sm[];  // [kWarps][TB][k]
  const RowLayout L = make_layout(g.k);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane / L.LPR, cl = lane % L.LPR;
  const int row0 = blockIdx.x * g.slab_rows;
  const int row1 = min(g.d, row0 + g.slab_rows);
  const float* x = io.x + (long long)io_slot(io) * io.x_step_stride;

  for (int t0 = 0; t0 < n_tokens; t0 += TB) {
    float acc[TB][VPL][8];
#pragma unroll
    for (int tt = 0; tt < TB; ++tt)
#pragma unroll
      for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[tt][v][e] = 0.f;

    for (int base = row0 + warp * L.RPP; base < row1; base += kWarps * L.RPP) {
      const int row = base + sub;
      if (row < row1) {
        float xv[TB];
#pragma unroll
        for (int tt = 0; tt < TB; ++tt)
          xv[tt] = (t0 + tt < n_tokens) ? __ldg(x + (size_t)(t0 + tt) * g.d + row) : 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          const int cv = cl + v * L.LPR;
          if (cv < L.KV) {
            float p8[8];
            load8<PF32>(g.P, (size_t)row * L.KV + cv, p8);
#pragma unroll
            for (int tt = 0; tt < TB; ++tt)
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[tt][v][e] = fmaf(p8[e], xv[tt], acc[tt][v][e]);
          }
        }
      }
    }
    // rows handled by different lane sub-groups of this warp
    for (int o = L.LPR; o < 32; o <<= 1) {
#pragma unroll
      for (int tt = 0; tt < TB; ++tt)
#pragma unroll
        for (int v = 0; v < VPL; ++v)
#pragma unroll
          for (int e = 0; e < 8; ++e)
            acc[tt][v][e] += __shfl_xor_sync(0xffffffffu, acc[tt][v][e], o);
    }
    if (sub == 0) {
#pragma unroll
      for (int tt = 0; tt < TB; ++tt)
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          const int cv = cl + v * L.LPR;
          if (cv < L.KV) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sm[(size_t)(warp * TB + tt) * g.k + cv * 8 + e] = acc[tt][v][e];
          }
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < TB * g.k; idx += kThreads) {
      const int tt = idx / g.k, j = idx - tt * g.k;
      if (t0 + tt < n_tokens) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += sm[(size_t)(w * TB + tt) * g.k + j];
        g.cpart[((size_t)blockIdx.x * g.B + t0 + tt) * g.k + j] = s;
      }
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(128) k_reduce_c(GroupParams g, int n_tokens) {
  const int j = blockIdx.x * 128 + threadIdx.x;
  const int t = blockIdx.y;
  if (j >= g.k || t >= n_tokens) return;
  float s = 0.f;
  for (int sl = 0; sl < g.n_slabs; ++sl) s += g.cpart[((size_t)sl * g.B + t) * g.k + j];
  g.c[(size_t)t * g.k + j] = s;
}

// dot[tt] = A[row][:] . c[tt][:] for the rows of one warp pass; every lane of
// the warp takes part (shuffles), invalid rows contribute zeros.
template <int VPL, bool AF32>
__device__ __forceinline__ void row_dot(const void* A, size_t row, bool valid, const RowLayout& L,
                                        int cl, const float (&c8)[TB][VPL][8], float (&dot)[TB]) {
#pragma unroll
  for (int tt = 0; tt < TB; ++tt) dot[tt] = 0.f;
  if (valid) {
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int cv = cl + v * L.LPR;
      if (cv < L.KV) {
        float a8[8];
        load8<AF32>(A, row * L.KV + cv, a8);
#pragma unroll
        for (int tt = 0; tt < TB; ++tt)
#pragma unroll
          for (int e = 0; e < 8; ++e) dot[tt] = fmaf(a8[e], c8[tt][v][e], dot[tt]);
      }
    }
  }
  for (int o = L.LPR >> 1; o > 0; o >>= 1) {
#pragma unroll
    for (int tt = 0; tt < TB; ++tt) dot[tt] += __shfl_xor_sync(0xffffffffu, dot[tt], o);
  }
}

template <int VPL>
__device__ __forceinline__ void load_c(const float* c, int k, int t0, int n_tokens,
                                       const RowLayout& L, int cl, float (&c8)[TB][VPL][8]) {
#pragma unroll
  for (int tt = 0; tt < TB; ++tt)
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int cv = cl + v * L.LPR;
      if (cv < L.KV && t0 + tt < n_tokens) {
        const float4* p = reinterpret_cast<const float4*>(c + (size_t)(t0 + tt) * k + cv * 8);
        float4 a = p[0], b = p[1];
        c8[tt][v][0] = a.x; c8[tt][v][1] = a.y; c8[tt][v][2] = a.z; c8[tt][v][3] = a.w;
        c8[tt][v][4] = b.x; c8[tt][v][5] = b.y; c8[tt][v][6] = b.z; c8[tt][v][7] = b.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) c8[tt][v][e] = 0.f;
      }
    }
}

template <int VPL, bool PF32>
__global__ void __launch_bounds__(kThreads)
k_residual_gate(GroupParams g, IoRef io, int n_tokens) {
  __shared__ float s_norm[kWarps][TB][2];
  __shared__ int s_last;
  const RowLayout L = make_layout(g.k);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane / L.LPR, cl = lane % L.LPR;
  const int row0 = blockIdx.x * g.slab_rows;
  const int row1 = min(g.d, row0 + g.slab_rows);
  const int slot = io_slot(io);
  const float* x = io.x + (long long)slot * io.x_step_stride;

  for (int t0 = 0; t0 < n_tokens; t0 += TB) {
    float c8[TB][VPL][8];
    load_c<VPL>(g.c, g.k, t0, n_tokens, L, cl, c8);
    float sr[TB], sx[TB];
#pragma unroll
    for (int tt = 0; tt < TB; ++tt) sr[tt] = sx[tt] = 0.f;
    for (int base = row0 + warp * L.RPP; base < row1; base += kWarps * L.RPP) {
      const int row = base + sub;
      const bool valid = row < row1;
      float dot[TB];
      row_dot<VPL, PF32>(g.P, (size_t)row, valid, L, cl, c8, dot);
      if (valid && cl == 0) {
#pragma unroll
        for (int tt = 0; tt < TB; ++tt) {
          if (t0 + tt < n_tokens) {
            const float xv = __ldg(x + (size_t)(t0 + tt) * g.d + row);
            const float rv = xv - dot[tt];
            g.r[(size_t)(t0 + tt) * g.d + row] = rv;
            sr[tt] = fmaf(rv, rv, sr[tt]);
            sx[tt] = fmaf(xv, xv, sx[tt]);
          }
        }
      }
    }
#pragma unroll
    for (int tt = 0; tt < TB; ++tt) {
      const float a = warp_sum(sr[tt]), b = warp_sum(sx[tt]);
      if (lane == 0) {
        s_norm[warp][tt][0] = a;
        s_norm[warp][tt][1] = b;
      }
    }
    __syncthreads();
    if (threadIdx.x < TB * 2) {
      const int tt = threadIdx.x >> 1, w = threadIdx.x & 1;
      if (t0 + tt < n_tokens) {
        float s = 0.f;
#pragma unroll
        for (int wp = 0; wp < kWarps; ++wp) s += s_norm[wp][tt][w];
        g.normpart[((size_t)blockIdx.x * g.B + t0 + tt) * 2 + w] = s;
      }
    }
    __syncthreads();
  }

  // The last slab to arrive sums the norm partials in slab order and decides.
  decide_gate_last_block(g, io, slot, n_tokens, g.normpart, g.n_slabs, gridDim.x, &s_last);
}

template <int VPL>
__global__ void __launch_bounds__(kThreads)
k_image_gemv(GroupParams g, IoRef io, int n_tokens) {
  const RowLayout L = make_layout(g.k);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane / L.LPR, cl = lane % L.LPR;
  const int rows_per_pass = kWarps * L.RPP;
  for (int t0 = 0; t0 < n_tokens; t0 += TB) {
    float c8[TB][VPL][8];
    load_c<VPL>(g.c, g.k, t0, n_tokens, L, cl, c8);
    for (int base = blockIdx.x * rows_per_pass + warp * L.RPP; base < g.O;
         base += gridDim.x * rows_per_pass) {
      const int row = base + sub;
      const bool valid = row < g.O;
      float dot[TB];
      row_dot<VPL, false>(g.WP, (size_t)row, valid, L, cl, c8, dot);
      if (valid && cl == 0) {
#pragma unroll
        for (int tt = 0; tt < TB; ++tt)
          if (t0 + tt < n_tokens) io.y[(size_t)(t0 + tt) * g.O + row] = dot[tt];
      }
    }
  }
}

// y[tok][a] (+)= W[a][:] . src[tok][:], one warp per output row, W streamed
// once per chunk of TB tokens.  kDense: every token, y overwritten, src = x.
// Otherwise only the fired tokens, y accumulated into, src = r.
template <bool kDense>
__global__ void __launch_bounds__(kThreads)
k_stream_gemv(GroupParams g, IoRef io, int n_tokens) {
  const int n = kDense ? n_tokens : *g.n_fired;
  if (n == 0) return;
  if (!kDense && g.tc_min_fired > 0 && n >= g.tc_min_fired) return;  // tensor-core path takes it
  const int slot = io_slot(io);
  const float* src = kDense ? io.x + (long long)slot * io.x_step_stride : g.r;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int DV = g.d / 8;
  if (kDense && blockIdx.x == 0) {
    unsigned char* gate = io.gate + (long long)slot * io.log_step_stride;
    for (int t = threadIdx.x; t < n_tokens; t += kThreads) gate[t] = 1;
  }
  for (int a = blockIdx.x * kWarps + warp; a < g.O; a += gridDim.x * kWarps) {
    int j = 0;
    while (j + 1 < g.n_maps && a >= g.off[j + 1]) ++j;
    const uint4* wrow = reinterpret_cast<const uint4*>(g.W[j] + (size_t)(a - g.off[j]) * g.d);
    for (int f0 = 0; f0 < n; f0 += TB) {
      int tok[TB];
      float acc[TB];
#pragma unroll
      for (int tt = 0; tt < TB; ++tt) {
        tok[tt] = (f0 + tt < n) ? (kDense ? f0 + tt : g.fired[f0 + tt]) : -1;
        acc[tt] = 0.f;
      }
      for (int v0 = lane; v0 < DV; v0 += 4 * kWarp) {
        uint4 w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int v = v0 + u * kWarp;
          w[u] = (v < DV) ? ld_stream(wrow + v) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int v = v0 + u * kWarp;
          if (v < DV) {
            float w8[8];
            unpack_bf16x8(w[u], w8);
#pragma unroll
            for (int tt = 0; tt < TB; ++tt) {
              if (tok[tt] >= 0) {
                const float4* rp =
                    reinterpret_cast<const float4*>(src + (size_t)tok[tt] * g.d + (size_t)v * 8);
                const float4 r0 = __ldg(rp), r1 = __ldg(rp + 1);
                float s = acc[tt];
                s = fmaf(w8[0], r0.x, s); s = fmaf(w8[1], r0.y, s);
                s = fmaf(w8[2], r0.z, s); s = fmaf(w8[3], r0.w, s);
                s = fmaf(w8[4], r1.x, s); s = fmaf(w8[5], r1.y, s);
                s = fmaf(w8[6], r1.z, s); s = fmaf(w8[7], r1.w, s);
                acc[tt] = s;
              }
            }
          }
        }
      }
#pragma unroll
      for (int tt = 0; tt < TB; ++tt) {
        const float s = warp_sum(acc[tt]);
        if (lane == 0 && tok[tt] >= 0) {
          float* yp = io.y + (size_t)tok[tt] * g.O + a;
          *yp = kDense ? s : (*yp + s);
        }
      }
    }
  }
}

__global__ void k_advance_step(int* step) {
  if (threadIdx.x == 0 && blockIdx.x == 0) *step = *step + 1;
}

// Algorithm 1 lines 1-4 on CUDA cores: c, r, norms, gate (and, with_image, line 5).
template <int VPL>
cudaError_t launch_vpl(const GroupParams& g, const IoRef& io, int n_tokens, cudaStream_t st,
                       int* n_launches, bool with_image = true) {
  const RowLayout L = make_layout(g.k);
  const size_t sm = (size_t)kWarps * TB * g.k * sizeof(float);
  cudaError_t e;
  if (g.p_f32) {
    e = cudaFuncSetAttribute(k_project_partial<VPL, true>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    k_project_partial<VPL, true><<<g.n_slabs, kThreads, sm, st>>>(g, io, n_tokens);
  } else {
    e = cudaFuncSetAttribute(k_project_partial<VPL, false>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    k_project_partial<VPL, false><<<g.n_slabs, kThreads, sm, st>>>(g, io, n_tokens);
  }
  k_reduce_c<<<dim3((g.k + 127) / 128, n_tokens), 128, 0, st>>>(g, n_tokens);
  if (g.p_f32)
    k_residual_gate<VPL, true><<<g.n_slabs, kThreads, 0, st>>>(g, io, n_tokens);
  else
    k_residual_gate<VPL, false><<<g.n_slabs, kThreads, 0, st>>>(g, io, n_tokens);
  *n_launches += 3;
  if (with_image) {
    const int rows_per_pass = kWarps * L.RPP;
    int grid = (g.O + rows_per_pass - 1) / rows_per_pass;
    if (grid > 148 * 8) grid = 148 * 8;
    k_image_gemv<VPL><<<grid, kThreads, 0, st>>>(g, io, n_tokens);
    *n_launches += 1;
  }
  return cudaGetLastError();
}

cudaError_t dispatch_vpl(const GroupParams& g, const IoRef& io, int n_tokens, cudaStream_t st,
                         int* n_launches, bool with_image) {
  switch (make_layout(g.k).VPL) {
    case 1: return launch_vpl<1>(g, io, n_tokens, st, n_launches, with_image);
    case 2: return launch_vpl<2>(g, io, n_tokens, st, n_launches, with_image);
    case 3: return launch_vpl<3>(g, io, n_tokens, st, n_launches, with_image);
    case 4: return launch_vpl<4>(g, io, n_tokens, st, n_launches, with_image);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_generic_forward(const GroupParams& g, const TmaMaps* tm, const IoRef& io,
                                   int n_tokens, cudaStream_t st, int* n_launches, ResidualLane* lane) {
  int dummy = 0;
  if (!n_launches) n_launches = &dummy;
  int grid = (g.O + kWarps - 1) / kWarps;
  if (grid > 148 * 8) grid = 148 * 8;
  if (g.flags & GSI_FLAG_DENSE) {
    if (tm && g.front_min_tokens > 0 && n_tokens >= g.front_min_tokens)
      return launch_dense_gemm_tc(g, *tm, io, n_tokens, st, n_launches);
    k_stream_gemv<true><<<grid, kThreads, 0, st>>>(g, io, n_tokens);
    *n_launches += 1;
    return cudaGetLastError();
  }
  cudaError_t e;
  const bool front = tm && g.front_min_tokens > 0 && n_tokens >= g.front_min_tokens;
  if (front) {
    e = launch_front_tc(g, *tm, io, n_tokens, st, n_launches);
  } else {
    e = dispatch_vpl(g, io, n_tokens, st, n_launches, true);
  }
  if (e != cudaSuccess) return e;
  if (!(g.flags & GSI_FLAG_STATIC_PROJECTION)) {
    if (front) {
      // every gated token goes through the tensor-core contraction; r is in rb already
      cudaStream_t sr = st;
      if (lane) {   // behind this group's gate, beside the next groups' projections
        if ((e = cudaEventRecord(lane->ev, st)) != cudaSuccess ||
            (e = cudaStreamWaitEvent(lane->stream, lane->ev, 0)) != cudaSuccess)
          return e;
        sr = lane->stream;
        lane->used = true;
      }
      e = launch_residual_gemm_tc(g, *tm, io, 1, true, n_tokens, sr, n_launches);
      if (e != cudaSuccess) return e;
    } else {
      k_stream_gemv<false><<<grid, kThreads, 0, st>>>(g, io, n_tokens);
      *n_launches += 1;
      if (tm && g.tc_min_fired > 0) {
        e = launch_residual_gemm_tc(g, *tm, io, g.tc_min_fired, false, n_tokens, st, n_launches);
        if (e != cudaSuccess) return e;
      }
    }
  }
  return cudaGetLastError();
}

cudaError_t launch_project_residual(const GroupParams& g, const IoRef& io, cudaStream_t st) {
  int n = 0;
  return dispatch_vpl(g, io, 1, st, &n, false);
}

cudaError_t launch_gated_gemv(const GroupParams& g, const IoRef& io, cudaStream_t st) {
  int grid = (g.O + kWarps - 1) / kWarps;
  if (grid > 148 * 8) grid = 148 * 8;
  k_stream_gemv<false><<<grid, kThreads, 0, st>>>(g, io, 1);
  return cudaGetLastError();
}

int generic_launch_count(const GroupParams& g, int n_tokens) {
  // (a tensor-core contraction with one split over the depth writes y itself: no kernel that adds partial sums)
  const int add = tc_splits(g.O, g.d) > 1 ? 1 : 0;
  if (g.flags & GSI_FLAG_DENSE)
    return (g.front_min_tokens > 0 && n_tokens >= g.front_min_tokens) ? 2 + add : 1;
  const bool stat = g.flags & GSI_FLAG_STATIC_PROJECTION;
  if (g.front_min_tokens > 0 && n_tokens >= g.front_min_tokens) return stat ? 4 : 5 + add;
  return 4 + (stat ? 0 : 1 + (g.tc_min_fired > 0 ? 2 + add : 0));
}

cudaError_t launch_advance_step(int* step, cudaStream_t st) {
  k_advance_step<<<1, 32, 0, st>>>(step);
  return cudaGetLastError();
}

// ---- image build: W_P = bf16(W P), fp32 accumulation -------------------------
namespace {
constexpr int IT = 64;   // tile of output rows / columns
constexpr int IK = 16;   // depth step

template <bool PF32>
__global__ void __launch_bounds__(256)
k_build_image(const uint16_t* __restrict__ W, const void* __restrict__ P, int o, int d, int k,
              uint16_t* __restrict__ WP) {
  __shared__ float As[IK][IT + 1];
  __shared__ float Bs[IK][IT];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int o0 = blockIdx.y * IT, k0 = blockIdx.x * IT;
  float acc[4][4] = {};
  for (int d0 = 0; d0 < d; d0 += IK) {
    for (int idx = threadIdx.x; idx < IT * IK; idx += 256) {
      const int m = idx / IK, kk = idx % IK;
      float v = 0.f;
      if (o0 + m < o && d0 + kk < d)
        v = __uint_as_float(((uint32_t)W[(size_t)(o0 + m) * d + d0 + kk]) << 16);
      As[kk][m] = v;
    }
    for (int idx = threadIdx.x; idx < IT * IK; idx += 256) {
      const int kk = idx / IT, n = idx % IT;
      float v = 0.f;
      if (d0 + kk < d && k0 + n < k) {
        const size_t at = (size_t)(d0 + kk) * k + k0 + n;
        if constexpr (PF32) v = reinterpret_cast<const float*>(P)[at];
        else v = __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(P)[at]) << 16);
      }
      Bs[kk][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < IK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = o0 + ty * 4 + i, n = k0 + tx * 4 + j;
      if (m < o && n < k) {
        __nv_bfloat16 h = __float2bfloat16_rn(acc[i][j]);
        WP[(size_t)m * k + n] = *reinterpret_cast<uint16_t*>(&h);
      }
    }
}
}  // namespace

cudaError_t launch_build_image(const void* W, const void* P, int o, int d, int k, bool p_f32,
                               void* WP, cudaStream_t st) {
  dim3 grid((k + IT - 1) / IT, (o + IT - 1) / IT);
  if (p_f32)
    k_build_image<true><<<grid, 256, 0, st>>>((const uint16_t*)W, P, o, d, k, (uint16_t*)WP);
  else
    k_build_image<false><<<grid, 256, 0, st>>>((const uint16_t*)W, P, o, d, k, (uint16_t*)WP);
  return cudaGetLastError();
}

}  // namespace gsi
