// One 128-row accumulator tile on the 5th-gen tensor cores, shared by the batched
// kernels: D[128 x N] (fp32, tensor memory) = A[128 x K] * B[N x K]^T with bf16
// operands that are both K-major in global memory.
//
//   A, B tiles (64 K-elements = 128 bytes per row and stage) go global -> shared by
//   cp.async, written in the 128-byte-swizzled K-major layout the descriptors name;
//   one thread issues tcgen05.mma; tcgen05.commit frees a stage through an mbarrier;
//   the caller reads D with tcgen05.ld and then releases the tensor memory.
//
// Every wait is bounded: a timeout makes tile_mma return false (uniformly for the
// block) and the caller reports it; the tensor memory is released in either case.
#pragma once

#include "gsi_common.cuh"

namespace gsi {
namespace umma {

constexpr int kTM = 128;          // rows of A per tile (tensor-memory lanes)
constexpr int kTK = 64;           // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int kThreads = 128;
constexpr int kABytes = kTM * kTK * 2;     // 16 KB
constexpr unsigned kSpin = 1u << 22;

template <int kStages, int kBRows>
struct Cfg {
  static constexpr int kBBytes = kBRows * kTK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kSmem = 1024 /*align slack*/ + kStages * kStageBytes + 256;
};

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
// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15])
      : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Runs the whole contraction of one tile: rows [0,128) of A (row stride lda
// elements), rows [0,N) of B (row stride ldb; operand row n is row b_rows[n] of B when
// b_rows, a table the block wrote before the call, is not null), K blocks
// [kb0, kb0+nloc) of 64 elements.  N is a multiple of 16 in [16, kBRows].  All kThreads threads of the
// block call it.  On return *tmem_out holds the tensor-memory base of D (lane =
// row, column = B row); the return value, the same for every thread, is false when a
// wait ran out of time.  With nloc == 0 nothing is accumulated and D is undefined.
// The caller must end with tile_release<kTmemCols>(*tmem_out).
template <int kStages, int kBRows, int kTmemCols>
__device__ __forceinline__ bool tile_mma(unsigned char* smem_raw, const uint16_t* A, size_t lda,
                                         const uint16_t* B, size_t ldb, const int* b_rows, int N,
                                         int kb0, int nloc, uint32_t* tmem_out) {
  using C = Cfg<kStages, kBRows>;
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bar_free = reinterpret_cast<uint64_t*>(smem + kStages * C::kStageBytes);  // [kStages]
  uint64_t* bar_done = bar_free + kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_done + 1);
  int* s_fail = reinterpret_cast<int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5;

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
  *tmem_out = tmem;

  // one stage: A tile 128 rows x 8 chunks of 16 B, B tile N rows x 8 chunks, both written
  // at chunk ^ (row & 7): the 128-byte swizzle the descriptors announce
  auto load_stage = [&](int kb, int stage) {
    unsigned char* sa = smem + stage * C::kStageBytes;
    unsigned char* sb = sa + kABytes;
    const size_t koff = (size_t)kb * kTK;   // elements
#pragma unroll
    for (int it = 0; it < (kTM * 8) / kThreads; ++it) {
      const int idx = it * kThreads + tid, row = idx >> 3, ch = idx & 7;
      cp_async16(s32(sa + row * 128 + ((ch ^ (row & 7)) << 4)), A + (size_t)row * lda + koff + ch * 8);
    }
    for (int idx = tid; idx < N * 8; idx += kThreads) {
      const int row = idx >> 3, ch = idx & 7;
      const int src = b_rows ? b_rows[row] : row;
      cp_async16(s32(sb + row * 128 + ((ch ^ (row & 7)) << 4)), B + (size_t)src * ldb + koff + ch * 8);
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
      const uint32_t a0 = s32(smem + stage * C::kStageBytes), b0 = a0 + kABytes;
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
  const bool mine = !*s_fail && mbar_wait(bar_done, 0);
  const bool done = __syncthreads_and(mine ? 1 : 0) != 0;   // the same answer for every thread
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  return done;
}

template <int kTmemCols>
__device__ __forceinline__ void tile_release(uint32_t tmem) {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if ((threadIdx.x >> 5) == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
}

}  // namespace umma
}  // namespace gsi
