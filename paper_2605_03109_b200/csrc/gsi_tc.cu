// Gated residual for MANY fired tokens as a dense contraction on the 5th-gen
// tensor cores (Eq. (3.2): y_t += W r_t for every gated token t of the batch).
//
// Swap-AB formulation: the accumulator tile is D[128 rows of W][N tokens], N the
// fired-token count padded to a multiple of 16 (16..64).  W is streamed exactly
// once per step; the contraction stays HBM-bound (<= 64 FLOP/B, far below the
// tensor ridge), the tensor pipe is only the means to stay on the HBM roofline
// once there are too many tokens for CUDA-core FMAs.
//
//   A (W tile, 128 x 64 bf16 per stage)   global -> shared by cp.async, written in the
//   B (R tile,   N x 64 bf16 per stage)   128-byte-swizzled K-major layout tcgen05 reads
//   D (128 lanes x N columns fp32)        tensor memory; tcgen05.mma, one issuing thread
//   epilogue                              tcgen05.ld -> registers -> partial-sum buffer
//
// Split-K over CTAs fills the machine for the narrow maps; partial sums are added
// to y in a fixed order by a second small kernel, so results are reproducible.
// Every wait is bounded; a timeout sets the status word, frees the tensor memory
// and returns.
#include "gsi_common.cuh"

namespace gsi {

namespace {

constexpr int kTM = 128;          // rows of W per CTA tile (tensor-memory lanes)
constexpr int kTK = 64;           // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int kStages = 6;
constexpr int kMaxN = 64;
constexpr int kThreadsTc = 128;
constexpr int kABytes = kTM * kTK * 2;     // 16 KB
constexpr int kBBytes = kMaxN * kTK * 2;   //  8 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTmemCols = 64;
constexpr unsigned kSpin = 1u << 22;
constexpr int kTcSmem = 1024 /*align slack*/ + kStages * kStageBytes + 256;

__device__ __forceinline__ uint32_t s32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(count));
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(s32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity) {
  for (unsigned it = 0; it < kSpin; ++it)
    if (mbar_try(b, parity)) return true;
  return false;
}

// Shared-memory matrix descriptor, K-major operand in the 128-byte swizzle:
// rows of 128 bytes, eight-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFFu);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                   // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset between eight-row groups
  d |= (uint64_t)1 << 46;                   // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                   // layout: 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   s32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15])
      : "r"(addr));
}

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

__global__ void __launch_bounds__(kThreadsTc, 1)
k_residual_gemm_tc(GroupParams g, int min_fired, int splits) {
  const int n_fired = *g.n_fired;
  if (n_fired < min_fired) return;            // the CUDA-core GEMV handles the few-token case
  const int N = (n_fired + 15) & ~15;         // 16..64

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bar_free = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);  // [kStages]
  uint64_t* bar_done = bar_free + kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_done + 1);
  int* s_fail = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x / splits, split = blockIdx.x % splits;
  const int row0 = tile * kTM;                 // first row of the concatenated maps
  int j = 0;
  while (j + 1 < g.n_maps && row0 >= g.off[j + 1]) ++j;
  const uint16_t* Wt = g.W[j] + (size_t)(row0 - g.off[j]) * g.d;   // tile never straddles maps
  const int nkb = g.d / kTK;
  const int kb0 = (int)((long long)nkb * split / splits), kb1 = (int)((long long)nkb * (split + 1) / splits);
  const int nloc = kb1 - kb0;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&bar_free[s], 1);
    mbar_init(bar_done, 1);
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     s32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  // one stage: A tile 128 rows x 8 chunks of 16 B, B tile N rows x 8 chunks, both written
  // at chunk ^ (row & 7): the 128-byte swizzle the descriptors announce
  auto load_stage = [&](int kb, int stage) {
    unsigned char* sa = smem + stage * kStageBytes;
    unsigned char* sb = sa + kABytes;
    const size_t koff = (size_t)kb * kTK;   // elements
#pragma unroll
    for (int it = 0; it < (kTM * 8) / kThreadsTc; ++it) {
      const int idx = it * kThreadsTc + tid, row = idx >> 3, ch = idx & 7;
      cp_async16(s32(sa + row * 128 + ((ch ^ (row & 7)) << 4)),
                 Wt + (size_t)row * g.d + koff + ch * 8);
    }
    for (int idx = tid; idx < N * 8; idx += kThreadsTc) {
      const int row = idx >> 3, ch = idx & 7;
      cp_async16(s32(sb + row * 128 + ((ch ^ (row & 7)) << 4)),
                 g.rb + (size_t)row * g.d + koff + ch * 8);
    }
  };

  for (int s = 0; s < kStages - 1; ++s) {
    if (s < nloc) load_stage(kb0 + s, s);
    cp_async_commit();
  }
  const uint32_t idesc = instr_desc(kTM, N);
  bool ok = true;
  for (int i = 0; i < nloc && ok; ++i) {
    const int stage = i % kStages;
    cp_async_wait<kStages - 2>();                                    // block i of this thread landed
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // ...and is visible to the tensor core
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a0 = s32(smem + stage * kStageBytes), b0 = a0 + kABytes;
#pragma unroll
      for (int k = 0; k < kTK / 16; ++k)   // 32 bytes further along K per instruction
        umma_bf16(tmem, smem_desc_sw128(a0 + k * 32), smem_desc_sw128(b0 + k * 32), idesc,
                  (i > 0 || k > 0) ? 1u : 0u);
      umma_commit(&bar_free[stage]);       // arrives when the tensor core has read this stage
    }
    // refill the stage block i-1 used with block i+kStages-1
    const int nb = i + kStages - 1;
    if (nb < nloc) {
      if (i >= 1) {
        const int ps = (i - 1) % kStages;
        if (!mbar_wait(&bar_free[ps], ((i - 1) / kStages) & 1)) {
          *s_fail = 1;
          ok = false;
        }
      }
      if (ok) load_stage(kb0 + nb, nb % kStages);
    }
    cp_async_commit();
  }
  cp_async_wait<0>();
  if (tid == 0) umma_commit(bar_done);
  __syncthreads();
  if (*s_fail || !mbar_wait(bar_done, 0)) {
    if (tid == 0) atomicExch(g.status, (int)GSI_ERR_TIMEOUT);
  } else if (nloc > 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // warp w owns tensor-memory lanes 32w..32w+31 = rows row0+32w+lane; 16 columns per load
    float* yp = g.ypart + ((size_t)split * kMaxN) * g.O + row0 + warp * 32 + lane;
    for (int c0 = 0; c0 < N; c0 += 16) {
      uint32_t v[16];
      tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 16; ++c)
        if (c0 + c < n_fired) yp[(size_t)(c0 + c) * g.O] = __uint_as_float(v[c]);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
}

// y[fired[n]][row] += sum over splits (fixed order)
__global__ void __launch_bounds__(256) k_add_partials(GroupParams g, IoRef io, int min_fired, int splits) {
  const int n = *g.n_fired;
  if (n < min_fired) return;
  const int t = blockIdx.y;
  if (t >= n) return;
  const int tok = g.fired[t];
  for (int row = blockIdx.x * 256 + threadIdx.x; row < g.O; row += gridDim.x * 256) {
    float s = 0.f;
    for (int sp = 0; sp < splits; ++sp) s += g.ypart[((size_t)sp * kMaxN + t) * g.O + row];
    io.y[(size_t)tok * g.O + row] += s;
  }
}

}  // namespace

int tc_splits(int O, int d) {
  const int tiles = O / kTM, nkb = d / kTK;
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

cudaError_t launch_residual_gemm_tc(const GroupParams& g, const IoRef& io, int min_fired,
                                    cudaStream_t st, int* n_launches) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_residual_gemm_tc,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int splits = tc_splits(g.O, g.d);
  k_pack_fired_bf16<<<dim3((g.d + 2047) / 2048, kMaxN), 256, 0, st>>>(g, min_fired);
  k_residual_gemm_tc<<<(g.O / kTM) * splits, kThreadsTc, kTcSmem, st>>>(g, min_fired, splits);
  k_add_partials<<<dim3((g.O + 1023) / 1024, g.B), 256, 0, st>>>(g, io, min_fired, splits);
  if (n_launches) *n_launches += 3;
  return cudaGetLastError();
}

}  // namespace gsi
