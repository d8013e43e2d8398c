// One 128-row accumulator tile on the 5th-gen tensor cores, shared by the batched
// kernels: D[128 x N] (fp32, tensor memory) = A[128 x K] * B[N x K]^T with bf16
// operands that are both K-major in global memory.
//
//   producer thread   TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) brings a
//                     stage = A box 128 rows x 64 K-elements + N/16 B boxes of 16 rows into
//                     shared memory and signals the stage's "full" mbarrier by byte count
//   MMA thread        waits "full", issues tcgen05.mma (accumulator in tensor memory),
//                     tcgen05.commit arrives on the stage's "empty" mbarrier
//   all four warps    wait for the final commit, read D with tcgen05.ld (lane = row)
//
// The two loops never meet at a block-wide barrier, so the stages in flight are limited
// by shared memory only.  Every wait is bounded: a timeout makes tile_mma return false
// (uniformly for the block) after a bounded wait for the copies still in flight; the
// caller reports it and releases the tensor memory in either case.
#pragma once

#include <cuda.h>   // CUtensorMap (type only; the encoder is looked up at run time)

#include "gsi_common.cuh"

namespace gsi {
namespace umma {

constexpr int kTM = 128;          // rows of A per tile (tensor-memory lanes)
constexpr int kTK = 64;           // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int kBBox = 16;         // rows per B box
constexpr int kThreads = 128;
constexpr int kABytes = kTM * kTK * 2;     // 16 KB
constexpr unsigned kSpin = 1u << 22;

template <int kStages, int kBRows>
struct Cfg {
  static constexpr int kBBytes = kBRows * kTK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kSmem = 1024 /*align slack*/ + kStages * kStageBytes + 256;
  static_assert(kStageBytes % 1024 == 0, "stage bases must keep the 1024-byte swizzle alignment");
};

__device__ __forceinline__ uint32_t s32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(b)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_only(uint64_t* b, uint32_t bytes) {   // no arrival
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(b)) : "memory");
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
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, unsigned spin = kSpin) {
  for (unsigned it = 0; it < spin; ++it)
    if (mbar_try(b, parity)) return true;
  return false;
}
// One box of a 2-D tensor map: x = first K element, y = first row.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(s32(bar))
      : "memory");
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

// Runs the whole contraction of one tile: rows [a_row0, a_row0+128) of the matrix behind
// map_a, rows [b_row0, b_row0+N) of the matrix behind map_b, K blocks [kb0, kb0+nloc)
// of 64 elements.  N is a multiple of 16 in [16, kBRows].  All kThreads threads of the
// block call it.  On return *tmem_out holds the tensor-memory base of D (lane = row,
// column = B row); the return value, the same for every thread, is false when a wait ran
// out of time.  With nloc == 0 nothing is accumulated and D is undefined.  The caller
// must end with tile_release<kTmemCols>(*tmem_out).
// run_count / run_min: if run_count is given, it is read after the wait on the previous
// kernel and the contraction runs only if *run_count >= run_min; otherwise the weight boxes
// already requested are allowed to land, *skipped is set and the function returns true.
template <int kStages, int kBRows, int kTmemCols>
__device__ __forceinline__ bool tile_mma(unsigned char* smem_raw, const CUtensorMap* map_a,
                                         int a_row0, const CUtensorMap* map_b, int b_row0, int N,
                                         int kb0, int nloc, uint32_t* tmem_out,
                                         const int* run_count = nullptr, int run_min = 0,
                                         bool* skipped = nullptr) {
  using C = Cfg<kStages, kBRows>;
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bar_full = reinterpret_cast<uint64_t*>(smem + kStages * C::kStageBytes);  // [kStages]
  uint64_t* bar_empty = bar_full + kStages;                                            // [kStages]
  uint64_t* bar_done = bar_empty + kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_done + 1);
  int* s_fail = reinterpret_cast<int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar_full[s], 1);
      mbar_init(&bar_empty[s], 1);
    }
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
  const uint32_t stage_bytes = (uint32_t)(kABytes + N * kTK * 2);
  // The A operand is a weight tile (set-up data, never written by the kernels of a call):
  // its first kStages boxes are requested before the wait on the previous kernel, whose
  // output only the B operand can be.  (The first kernel of every chain of dependent
  // launches waits BEFORE it lets its successor start, so nothing launched ahead of the
  // chain can still be writing weights.)
  if (tid == 0) {
    for (int i = 0; i < nloc && i < kStages; ++i) {
      mbar_expect_tx_only(&bar_full[i], (uint32_t)kABytes);   // the arrival comes with the B boxes
      tma_load_2d(s32(smem + i * C::kStageBytes), map_a, (kb0 + i) * kTK, a_row0, &bar_full[i]);
    }
  }
  pdl_wait();   // the B operand may come from the previous kernel of the stream
  if (run_count && *run_count < run_min) {   // the same answer for every thread
    if (tid == 0) {
      for (int i = 0; i < nloc && i < kStages; ++i) {
        mbar_arrive(&bar_full[i]);
        (void)mbar_wait(&bar_full[i], 0);   // the requested boxes land before the block exits
      }
    }
    __syncthreads();
    if (skipped) *skipped = true;
    return true;
  }

  if (warp == 0) {
    if (lane == 0) {   // producer
      for (int i = 0; i < nloc; ++i) {
        const int stage = i % kStages;
        const uint32_t sa = s32(smem + stage * C::kStageBytes), sb = sa + kABytes;
        const int x = (kb0 + i) * kTK;
        if (i >= kStages) {
          if (!mbar_wait(&bar_empty[stage], ((i / kStages) - 1) & 1)) {
            *s_fail = 1;
            break;
          }
          mbar_expect_tx(&bar_full[stage], stage_bytes);
          tma_load_2d(sa, map_a, x, a_row0, &bar_full[stage]);
        } else {
          mbar_expect_tx(&bar_full[stage], stage_bytes - (uint32_t)kABytes);   // A is on its way
        }
        for (int j = 0; j < N / kBBox; ++j)
          tma_load_2d(sb + j * (kBBox * kTK * 2), map_b, x, b_row0 + j * kBBox, &bar_full[stage]);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {   // MMA issuer
      const uint32_t idesc = instr_desc(kTM, N);
      bool ok = true;
      for (int i = 0; i < nloc; ++i) {
        const int stage = i % kStages;
        if (!mbar_wait(&bar_full[stage], (i / kStages) & 1)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a0 = s32(smem + stage * C::kStageBytes), b0 = a0 + kABytes;
#pragma unroll
        for (int k = 0; k < kTK / 16; ++k)   // 32 bytes further along K per instruction
          umma_bf16(tmem, smem_desc_sw128(a0 + k * 32), smem_desc_sw128(b0 + k * 32), idesc,
                    (i > 0 || k > 0) ? 1u : 0u);
        umma_commit(&bar_empty[stage]);      // arrives when the tensor core has read this stage
      }
      if (ok) umma_commit(bar_done);
      else *s_fail = 1;
    }
    __syncwarp();
  }
  // Everyone: the accumulator is complete when the last commit arrives.  Warps 2 and 3
  // come straight here and poll while the pipeline runs.
  bool mine = mbar_wait(bar_done, 0, kSpin * 8);
  if (*reinterpret_cast<volatile int*>(s_fail)) mine = false;
  const bool done = __syncthreads_and(mine ? 1 : 0) != 0;   // the same answer for every thread
  if (!done && tid == 0) {
    // copies issued but not consumed: give them a bounded time to land before the block exits
    for (int s = 0; s < kStages && s < nloc; ++s) {
      const int last = ((nloc - 1 - s) / kStages) * kStages + s;   // last block that used stage s
      (void)mbar_wait(&bar_full[s], (last / kStages) & 1, 1u << 16);
    }
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  return done;
}

// fp32 operands enter the batched kernels as three bf16 terms in operand rows 3t, 3t+1,
// 3t+2 (t = token): this adds the three columns of 16 tokens, columns 48q .. 48q+47 of
// this thread's tensor-memory lane.
__device__ __forceinline__ void sum3_tokens16(uint32_t tmem_lane, int q, float (&s)[16]) {
  uint32_t v[3][16];
#pragma unroll
  for (int i = 0; i < 3; ++i) tmem_ld16(tmem_lane + 48 * q + 16 * i, v[i]);
  tmem_ld_wait();
#pragma unroll
  for (int tt = 0; tt < 16; ++tt) {
    const int c = 3 * tt;
    s[tt] = (__uint_as_float(v[c / 16][c % 16]) + __uint_as_float(v[(c + 1) / 16][(c + 1) % 16])) +
            __uint_as_float(v[(c + 2) / 16][(c + 2) % 16]);
  }
}
// Operand rows of n tokens, rounded up to the 16-row boxes.
__host__ __device__ __forceinline__ int term_rows(int n_tokens) { return (3 * n_tokens + 15) & ~15; }

template <int kTmemCols>
__device__ __forceinline__ void tile_release(uint32_t tmem) {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if ((threadIdx.x >> 5) == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
}

}  // namespace umma

// Tensor maps of one layer (host-encoded at set-up, passed to the kernels by value as a
// __grid_constant__ parameter).  A operands use boxes of 128 rows, B operands of 16 rows;
// every box is 64 K-elements wide with the 128-byte swizzle.
struct alignas(64) TmaMaps {
  CUtensorMap w[GSI_MAX_MAPS];   // W_j [d_out_j][d]
  CUtensorMap p;                 // P   [d][k]
  CUtensorMap pt;                // P^T [k][d]
  CUtensorMap wp;                // W_P [O][k]
  CUtensorMap xb;                // terms of x [rows][d]   (B operand)
  CUtensorMap cb;                // terms of c [rows][k]   (B operand)
  CUtensorMap rb;                // residuals  [65][d]     (B operand)
};

}  // namespace gsi
