// Persistent decode-step kernel: every group of the stack in ONE launch.
//
// One CTA per SM.  Each CTA owns a fixed slab of rows of every basis P and of
// every (concatenated) image W_P.  A producer warp streams those slabs from HBM
// into a ring of shared-memory slots with bulk async copies, in program order
// and independent of the data-dependent steps (weight addresses never depend
// on x), so the next group's weights arrive while the current group waits on
// its cross-CTA exchanges.  Fifteen consumer warps run Algorithm 1 per group (two
// consecutive groups declared independent share a phase on two parts of the grid):
//
//   pass 1     partial c = P_slab^T x_slab                     (line 1)
//   exchange 1 c = sum over CTAs, by 64-bit fixed-point atomics whose words
//              also count arrivals (no separate flag, no fence, order-free and
//              therefore bit-reproducible)
//   pass 2     r_slab = x_slab - P_slab c, partial ||r||^2      (lines 2-3)
//   exchange 2 every CTA publishes its partial ||r||^2 as one 32-bit word, the sign
//              bit carrying the parity of the launch (relaxed store: the word
//              validates itself, every launch rewrites every word), as soon as its
//              residual rows are done ...
//   image      y_rows = W_P,rows c                              (line 5)
//              ... and collects the words after its image rows, so the exchange
//              runs under them; every CTA sums the words in a fixed order and
//              takes the same gate decision                     (line 4)
//   gated      y_rows += W_rows r, W streamed with 256-bit loads, then a grid
//              barrier                                          (Eq. (3.2))
//
// Every wait is bounded; a wait that gives up records GSI_ERR_TIMEOUT in the
// status word, the CTA drains its copies in flight and returns.
//
// This header holds the kernel; every build of it (with or without the pair logic, for any
// rank or for rank 256 only) is compiled in a translation unit of its own.
#pragma once

#include <cstdio>
#include <cstdlib>

#include "gsi_common.cuh"
#include "gsi_persistent.cuh"

namespace gsi {

namespace {

constexpr int kNW = kPersistConsumerWarps;
constexpr int kNC = kNW * 32;               // consumer threads
constexpr int kThreadsP = kNC + 32;         // + producer warp
constexpr int kSlots = 10;
constexpr int kChunk = 16384;
constexpr int kSlice = 4096;                // columns of W per staged slice of r
constexpr int kWLoads = 4;                  // 256-bit loads per lane in flight in the W stream
constexpr unsigned kSpinLimit = 1u << 22;
constexpr int kCountShift = 54;

// shared memory map (bytes)
constexpr int kXBatch = 5;           // float4 loads of x in flight per thread
constexpr int kOffBar = 0;          // full[kSlots], empty[kSlots]
constexpr int kOffMisc = 256;       // abort flag, scalars
constexpr int kOffX = 512;          // x of this CTA's basis rows      (kPersistMaxPRows floats)
constexpr int kOffC = 1536;         // c                                (512 floats)
constexpr int kOffVals = 3584;      // exchange-2 values                (256 floats)
constexpr int kOffDesc = 4608;      // 4 group descriptors, 512 B each (this phase's and the next's)
constexpr int kDescSlots = 4;
constexpr int kOffRed = kOffDesc + kDescSlots * 512;   // cross-warp scratch (kNW*512 floats)
constexpr int kOffRq = kOffRed + kNW * 512 * 4;   // staged r, 4 interleaved quarters (16 KB)
constexpr int kOffYacc = kOffRq + 16384;          // per-row accumulators (kPersistMaxORows floats)
constexpr int kOffRing = ((kOffYacc + kPersistMaxORows * 4 + 1023) / 1024) * 1024;
constexpr int kSmemBytes = kOffRing + kSlots * kChunk;
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 CTA");
static_assert(sizeof(PersistGroup) <= 512 && sizeof(PersistGroup) % 4 == 0, "descriptor slot");
static_assert(kOffC - kOffX >= kPersistMaxPRows * 4, "x slab");
constexpr int kDescWords = (int)(sizeof(PersistGroup) / 4);

struct Misc {
  int abort;
  int gate;
  float amax;
  float sum2;
  int nonfinite;
  float sr;
  int deposits;   // warps that have handed in their ||r||^2 partial in this phase
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; gives up when the limit is reached or another thread aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort) {
  for (unsigned it = 0; it < kSpinLimit; ++it) {
    if (mbar_try(b, parity)) return true;
    if ((it & 1023u) == 1023u && *abort) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void csync() {  // consumer warps only
  asm volatile("bar.sync 1, %0;" ::"n"(kNC) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed_u32(unsigned* p, unsigned v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_relaxed_u32(unsigned* p, unsigned v) {
  asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void ld256_stream(const void* p, uint32_t (&v)[8]) {
  asm volatile(
      "ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7])
      : "l"(p));
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

__device__ __forceinline__ void fail(const PersistParams& p, Misc* misc) {
  misc->abort = 1;
  atomicExch(p.status, (int)GSI_ERR_TIMEOUT);
}

// Optional cycle trace of CTA 0 (sections of the per-group pipeline, summed
// over groups); p.trace == nullptr disables it.
struct Trace {
  unsigned long long* out;
  long long t;
  __device__ __forceinline__ void start(const PersistParams& p) {
    out = (threadIdx.x == 0 && p.trace) ? p.trace + (size_t)blockIdx.x * 16 : nullptr;
    if (out) t = clock64();
  }
  __device__ __forceinline__ void mark(int section) {
    if (out) {
      const long long now = clock64();
      out[section] += (unsigned long long)(now - t);
      t = now;
    }
  }
};


struct Slab {
  int p0, p1;  // basis rows owned by this CTA
  int o0, o1;  // rows of the concatenated maps owned by this CTA (image rows and W rows)
};
__device__ __forceinline__ Slab slab_of(const PersistGroup& g, int cta) {
  Slab s;
  s.p0 = min(g.d, cta * g.p_rows);
  s.p1 = min(g.d, s.p0 + g.p_rows);
  s.o0 = min(g.O, cta * g.o_rows);
  s.o1 = min(g.O, s.o0 + g.o_rows);
  return s;
}

// ------------------------------------------------------------------ producer
__device__ void producer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kSlots;
  unsigned char* ring = smem + kOffRing;
  volatile int* abort = &misc->abort;
  unsigned n = 0;
  for (int gi = 0; gi < p.n_groups && !*abort; ++gi) {
    const PersistGroup& g = p.groups[gi];
    if (g.flags & GSI_FLAG_DENSE) continue;
    const int lc = (int)blockIdx.x - g.cta0;
    if (lc < 0 || lc >= g.ncta) continue;   // its partner's share of the grid
    const Slab s = slab_of(g, lc);
    const int rc = kChunk / (g.k * 2);
    for (int part = 0; part < 2; ++part) {
      const int a = part ? s.o0 : s.p0, b = part ? s.o1 : s.p1;
      const uint16_t* base = part ? g.WP : g.P;
      for (int r = a; r < b; r += rc) {
        const int rows = min(rc, b - r);
        const unsigned slot = n % kSlots, ph = (n / kSlots) & 1u;
        if (!mbar_wait(&empty[slot], ph ^ 1u, abort)) {
          if (!*abort) fail(p, misc);
          goto drain;
        }
        const uint32_t bytes = (uint32_t)rows * g.k * 2;
        mbar_expect_tx(&full[slot], bytes);
        bulk_g2s(ring + (size_t)slot * kChunk, base + (size_t)r * g.k, bytes, &full[slot]);
        ++n;
      }
    }
  }
drain:
  // Every copy issued must have landed before the CTA may give up its shared
  // memory: wait (bounded) for the last kSlots chunks.
  {
    const unsigned first = n > (unsigned)kSlots ? n - kSlots : 0;
    for (unsigned c = first; c < n; ++c) {
      const unsigned slot = c % kSlots, ph = (c / kSlots) & 1u;
      for (unsigned it = 0; it < kSpinLimit; ++it)
        if (mbar_try(&full[slot], ph)) break;
    }
  }
}

// ------------------------------------------------------------------ consumer
// Lane layout over a row of k bf16: KV = k/8 vectors, LPR = min(32, KV) lanes
// per row, RPP = 32/LPR rows per warp pass, VPL = KV/LPR vectors per lane.
struct Ctx {
  int step, slot_io;
  int len;     // groups in the phase just run (1, or 2 for a pair)
  unsigned parity, tag;
  unsigned n;  // ring sequence number, advances exactly as in producer()
  Trace tr;
};

// ---- consumer building blocks.  The per-group code below is executed once per
// group and is deliberately compact (no templates, shifts instead of divisions,
// the rarely-taken gated residual out of line): the per-group loop has to stay
// resident in the SM's instruction cache, a loop that does not is bound by
// instruction fetch, not by memory.

// Sum eight per-lane row partials across the LPR = 1<<lpr_log2 lanes (8, 16 or
// 32) that share the rows.  Halving exchange: each level sends half of the
// values to the partner lane, so eight rows cost 4+2+1 shuffles plus
// log2(LPR/8) for the tail instead of 8*log2(LPR).  On return the lanes with
// cl % (LPR/8) == 0 hold the total of row cl / (LPR/8).
__device__ __forceinline__ float reduce8(float (&v)[8], int cl, int LPR) {
  int m = LPR >> 1;
  {
    const bool up = cl & m;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = up ? v[i] : v[i + 4];
      const float recv = __shfl_xor_sync(0xffffffffu, send, m);
      v[i] = (up ? v[i + 4] : v[i]) + recv;
    }
  }
  m >>= 1;
  {
    const bool up = cl & m;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = up ? v[i] : v[i + 2];
      const float recv = __shfl_xor_sync(0xffffffffu, send, m);
      v[i] = (up ? v[i + 2] : v[i]) + recv;
    }
  }
  m >>= 1;
  {
    const bool up = cl & m;
    const float send = up ? v[0] : v[1];
    const float recv = __shfl_xor_sync(0xffffffffu, send, m);
    v[0] = (up ? v[1] : v[0]) + recv;
  }
#pragma unroll 1
  for (m >>= 1; m > 0; m >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], m);
  return v[0];
}

struct Geo {       // lane geometry of one group (k a power of two, 64..512)
  int KV;          // 16-byte vectors per row
  int lpr_log2;    // log2(lanes per row), lanes per row = min(32, KV)
  int vpl;         // vectors per lane (1, or 2 for k = 512)
  int rc_log2;     // log2(rows per 16 KB chunk)
  int sub, cl;     // this lane: row sub-group and column lane
};

// Two-wide fp32 FMA of sm_100: one instruction for a pair of bf16 weights.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ unsigned long long bf16x2_to_f32x2(uint32_t w) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(w << 16), "r"(w & 0xFFFF0000u));
  return r;
}
__device__ __forceinline__ void fma2(unsigned long long& acc, unsigned long long a,
                                     unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ float sum2(unsigned long long v) {
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
  return lo + hi;
}

// out[i] = tile[row0 + i][:] . c   for eight rows, this lane's share of the columns
__device__ __forceinline__ void dot8(const uint4* tile, const float* s_c, const Geo& q, int row0,
                                     int rows, float (&v)[8]) {
  unsigned long long acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0ull;
  const int LPR = 1 << q.lpr_log2;
#pragma unroll 1
  for (int u = 0; u < q.vpl; ++u) {
    const int cv = q.cl + u * LPR;
    const float4 ca = *reinterpret_cast<const float4*>(s_c + cv * 8);
    const float4 cb = *reinterpret_cast<const float4*>(s_c + cv * 8 + 4);
    const unsigned long long c0 = pack2(ca.x, ca.y), c1 = pack2(ca.z, ca.w);
    const unsigned long long c2 = pack2(cb.x, cb.y), c3 = pack2(cb.z, cb.w);
    // rows past the end of the slab read the last row again (no branch: the eight loads
    // and FMA chains interleave); the caller drops their results
#pragma unroll
    for (int h = 0; h < 8; h += 4) {   // four rows at a time: eight would not fit the registers
      uint4 w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = tile[max(min(row0 + h + i, rows - 1), 0) * q.KV + cv];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        fma2(acc[h + i], bf16x2_to_f32x2(w[i].x), c0);
        fma2(acc[h + i], bf16x2_to_f32x2(w[i].y), c1);
        fma2(acc[h + i], bf16x2_to_f32x2(w[i].z), c2);
        fma2(acc[h + i], bf16x2_to_f32x2(w[i].w), c3);
      }
      asm volatile("" ::: "memory");
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = sum2(acc[i]);
}

// 2^e as a double, e in the normal range
__device__ __forceinline__ double pow2d(int e) { return __hiloint2double((1023 + e) << 20, 0); }

// Grid-wide arrival counter: add one, wait (bounded) until `target` arrived.
__device__ __forceinline__ bool grid_arrive_wait(unsigned* ctr, unsigned target,
                                                 const PersistParams& p, Misc* misc) {
  volatile int* abort = &misc->abort;
  red_relaxed_u32(ctr, 1u);
  unsigned it = 0;
  while (ld_relaxed_u32(ctr) < target) {
    if (++it > kSpinLimit || *abort) {
      if (!*abort) fail(p, misc);
      return false;
    }
  }
  return true;
}

// ---- F. gated residual: y_rows (+)= W_rows . src (src = r, or x for the dense
// baseline).  Out of line: most groups skip it.
__device__ __noinline__ void gated_pass(const PersistGroup& g, const Slab& s, const float* src,
                                        float* y, bool dense, unsigned char* smem) {
  float4* s_rq = reinterpret_cast<float4*>(smem + kOffRq);
  float* s_yacc = reinterpret_cast<float*>(smem + kOffYacc);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rows = s.o1 - s.o0;
  const int nsl = (g.d + kSlice - 1) / kSlice;
#pragma unroll 1
  for (int sl = 0; sl < nsl; ++sl) {
    const int c0 = sl * kSlice, cols = min(kSlice, g.d - c0), nv = cols >> 4;
    csync();
#pragma unroll 1
    for (int v = tid; v < nv; v += kNC) {
      const float4* sp = reinterpret_cast<const float4*>(src + c0 + v * 16);
#pragma unroll
      for (int q = 0; q < 4; ++q) s_rq[q * 256 + v] = __ldcg(sp + q);
    }
    csync();
    auto row_ptr = [&](int rw) -> const uint16_t* {
      const int a = s.o0 + rw;
      int j = 0;
      while (j + 1 < g.n_maps && a >= g.off[j + 1]) ++j;
      return g.W[j] + (size_t)(a - g.off[j]) * g.d + c0;
    };
    // kWLoads x 256-bit loads per lane are in flight before the first FMA.
#pragma unroll 1
    for (int rw = warp; rw < rows; rw += kNW) {
      const uint16_t* wrow = row_ptr(rw);
      unsigned long long acc2 = 0ull;  // two fp32 partial sums (two-wide FMA)
#pragma unroll 1
      for (int v0 = lane; v0 < nv; v0 += kWLoads * 32) {
        uint32_t w[kWLoads][8];
#pragma unroll
        for (int u = 0; u < kWLoads; ++u) {
          const int v = v0 + u * 32;
          if (v < nv) ld256_stream(wrow + (size_t)v * 16, w[u]);
        }
#pragma unroll
        for (int u = 0; u < kWLoads; ++u) {
          const int v = v0 + u * 32;
          if (v < nv) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 rr = s_rq[q * 256 + v];
              fma2(acc2, bf16x2_to_f32x2(w[u][2 * q]), pack2(rr.x, rr.y));
              fma2(acc2, bf16x2_to_f32x2(w[u][2 * q + 1]), pack2(rr.z, rr.w));
            }
          }
        }
      }
      const float acc = warp_sum(sum2(acc2));
      if (lane == 0) s_yacc[rw] = (sl == 0 ? 0.f : s_yacc[rw]) + acc;
    }
  }
  __syncwarp();
#pragma unroll 1
  for (int rw = warp; rw < rows; rw += kNW) {
    if (lane == 0) {
      float* yp = y + s.o0 + rw;
      *yp = dense ? s_yacc[rw] : (__ldcg(yp) + s_yacc[rw]);
    }
  }
}

// Make the next group's activations L2-resident while this group runs (a real
// pipeline would find them there, written by the preceding operator).
__device__ __forceinline__ void prefetch_next_x(const PersistGroup& gn, int slot_io, int n_tokens,
                                                int who = 0) {
  if ((int)blockIdx.x == who) {
    const char* xn = reinterpret_cast<const char*>(gn.x + (long long)slot_io * gn.x_step_stride);
    const int lines = (gn.d * 4 * n_tokens + 127) >> 7;
    for (int l = threadIdx.x; l < lines; l += kNC) prefetch_l2(xn + (size_t)l * 128);
  }
}

// One group.  Returns false when the CTA must stop (a wait gave up).
// kPairs = false compiles the pair logic out: stacks without concurrent groups run a smaller
// loop (the per-phase code has to stay resident in the instruction cache).  kK != 0 is a
// build for stacks whose groups all have rank kK (shifts, strides and loop bounds become
// constants); kK = 0 reads the rank from the descriptor.
template <bool kPairs, int kK>
__device__ bool group_phase(const PersistParams& p, unsigned char* smem, Misc* misc, Ctx& ctx,
                            int gi) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kSlots;
  float* s_x = reinterpret_cast<float*>(smem + kOffX);
  float* s_c = reinterpret_cast<float*>(smem + kOffC);
  float* s_vals = reinterpret_cast<float*>(smem + kOffVals);
  float* s_red = reinterpret_cast<float*>(smem + kOffRed);
  unsigned char* ring = smem + kOffRing;
  volatile int* abort = &misc->abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int slot_io = ctx.slot_io;
  const unsigned parity = ctx.parity, tag = ctx.tag;
  unsigned& n = ctx.n;
  Trace& tr = ctx.tr;

  // The descriptors of this phase (one group, or a pair of independent groups that split
  // the grid) were staged in shared memory one phase ago, descriptor i in slot i % 4;
  // stage the next phase's now.
  auto desc = [&](int i) -> const PersistGroup& {
    return *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (i & (kDescSlots - 1)) * 512);
  };
  const PersistGroup& gA = desc(gi);
  const int len = kPairs ? gA.phase_len : 1, next_len = kPairs ? gA.next_len : min(gA.next_len, 1);
  const PersistGroup& gB = desc(gi + len - 1);   // gA itself when the group is alone
  const bool second = kPairs && cta >= gA.cta0 + gA.ncta;  // never when alone: its share is the whole grid
  const PersistGroup& g = second ? gB : gA;      // the group whose fast path this CTA runs
  const int gi_mine = gi + (second ? 1 : 0);
  const int lc = cta - g.cta0;                   // index within the group's share of the grid
  const PersistGroup& g_next = desc(gi + len);
  const bool has_next = next_len > 0;
  ctx.len = len;
  uint32_t desc_word = 0;  // one word of the next descriptors, in flight during section A
  if (tid < next_len * kDescWords)
    desc_word = __ldg(reinterpret_cast<const uint32_t*>(p.groups + gi + len) + tid);
  uint32_t* const desc_dst =
      reinterpret_cast<uint32_t*>(smem + kOffDesc +
                                  ((gi + len + (tid >= kDescWords ? 1 : 0)) & (kDescSlots - 1)) * 512) +
      (tid >= kDescWords ? tid - kDescWords : tid);

  const Slab s = slab_of(g, lc);
  const float* x = g.x + (long long)slot_io * g.x_step_stride + (size_t)p.token * g.d;
  float* const y_tok = g.y + (size_t)p.token * g.O;   // this launch's token
  const bool dense = g.flags & GSI_FLAG_DENSE;
  const bool zeroer = lc == gi_mine % g.ncta;  // this CTA clears the group's counters for the next launch
  int gate = 1, gate_other = 0;
  const float* rsrc = x;

  if (!dense) {
    const int k = kK ? kK : g.k;   // a build for one rank folds the whole lane geometry
    Geo q;
    q.KV = k >> 3;
    q.lpr_log2 = q.KV >= 32 ? 5 : 31 - __clz(q.KV);
    q.vpl = q.KV > 32 ? q.KV >> 5 : 1;
    q.rc_log2 = 31 - __clz(kChunk / 2) - (31 - __clz(k));  // rows per chunk = 8192 / k
    const int LPR = 1 << q.lpr_log2;
    q.sub = lane >> q.lpr_log2;
    q.cl = lane & (LPR - 1);
    const int rpp_log2 = 5 - q.lpr_log2;  // rows per warp pass
    const int rc = 1 << q.rc_log2;
    const int n_contrib = (g.d + g.p_rows - 1) / g.p_rows;  // CTAs that own basis rows
    unsigned long long* acc = g.acc_c + (size_t)parity * k * kAccStride;
    const int prow = s.p1 - s.p0, orow = s.o1 - s.o0;
    const int pchunks = (prow + rc - 1) >> q.rc_log2, ochunks = (orow + rc - 1) >> q.rc_log2;

    // ---- A. statistics of x (every CTA, the whole vector): max |x|, sum x^2,
    //      non-finite flag; x of this CTA's basis rows goes to shared memory.
    float amax = 0.f, sum2 = 0.f;
    const int d4 = g.d >> 2;
#pragma unroll 1
    for (int i0 = tid; i0 < d4; i0 += kXBatch * kNC) {   
      float4 v[kXBatch];
#pragma unroll
      for (int u = 0; u < kXBatch; ++u) {
        const int i4 = i0 + u * kNC;
        v[u] = i4 < d4 ? __ldcg(reinterpret_cast<const float4*>(x) + i4) : make_float4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kXBatch; ++u) {
        amax = fmaxf(fmaxf(amax, fmaxf(fabsf(v[u].x), fabsf(v[u].y))),
                     fmaxf(fabsf(v[u].z), fabsf(v[u].w)));
        sum2 = fmaf(v[u].x, v[u].x, sum2);
        sum2 = fmaf(v[u].y, v[u].y, sum2);
        sum2 = fmaf(v[u].z, v[u].z, sum2);
        sum2 = fmaf(v[u].w, v[u].w, sum2);
      }
    }
    if (tid < prow) s_x[tid] = __ldcg(x + s.p0 + tid);
    if (tid < next_len * kDescWords) *desc_dst = desc_word;
    tr.mark(0);
    // fmaxf drops NaN, the sum keeps it (and overflows to inf for huge inputs):
    // sum2 - sum2 is non-zero exactly when some x_i is NaN or inf (or x^2 overflowed)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      sum2 += __shfl_xor_sync(0xffffffffu, sum2, o);
    }
    if (lane == 0) {   // s_vals is idle until this group's exchange 2
      s_vals[warp * 2 + 0] = amax;
      s_vals[warp * 2 + 1] = sum2;
    }
    if (tid == 0) misc->deposits = 0;
    if (zeroer) {  // clear what the NEXT launch will accumulate into
#pragma unroll 1
      for (int j = tid; j < k; j += kNC)
        g.acc_c[((size_t)(parity ^ 1u) * k + j) * kAccStride] = 0ull;
      if (tid < 3) g.bar[2 * tid + (parity ^ 1u)] = 0u;
    }
    csync();
    if (has_next) prefetch_next_x(g_next, slot_io, p.n_tokens);
    if (next_len == 2) prefetch_next_x(desc(gi + len + 1), slot_io, p.n_tokens, 1);
    {  // every thread folds the warp partials in the same order
      float a = 0.f, t = 0.f;
#pragma unroll
      for (int w = 0; w < kNW; ++w) {
        a = fmaxf(a, s_vals[w * 2]);
        t += s_vals[w * 2 + 1];
      }
      amax = a;
      sum2 = t;
    }
    const bool nonfinite = !(sum2 - sum2 == 0.f);
    tr.mark(1);
    // fixed-point scale: |partial c_j| <= amax * rows * max|P| < 2^e
    double scale = 0.0, inv_scale = 0.0;
    {
      const float bound = amax * (float)g.p_rows * g.pmax;
      if (!nonfinite && bound > 0.f && bound < 3.0e38f) {
        const int e = max((int)((__float_as_uint(bound) >> 23) & 0xFFu), 1) - 126;
        scale = pow2d(43 - e);
        inv_scale = pow2d(e - 43);
      }
    }

    // ---- B. pass 1: partial c over this CTA's basis rows
    const unsigned n_p0 = n;
    bool ok = true;
    {  // the basis chunks of this group: one per lane, all waits in flight together
      bool mine_ok = true;
      if (lane < pchunks) {
        const unsigned seq = n_p0 + lane;
        mine_ok = mbar_wait(&full[seq % kSlots], (seq / kSlots) & 1u, abort);
      }
      ok = __all_sync(0xffffffffu, mine_ok);
    }
    tr.mark(2);
#pragma unroll 1
    for (int u = 0; u < q.vpl; ++u) {
      const int cv = q.cl + u * LPR;
      float a8[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) a8[e] = 0.f;
#pragma unroll 1
      for (int ci = 0; ci < pchunks; ++ci) {
        if (!ok) break;
        const unsigned sl = (n_p0 + ci) % kSlots;
        const uint4* tile = reinterpret_cast<const uint4*>(ring + (size_t)sl * kChunk);
        const int r_lo = ci << q.rc_log2, rows = min(rc, prow - r_lo);
#pragma unroll 1
        for (int row = (warp << rpp_log2) + q.sub; row < rows; row += kNW << rpp_log2) {
          const float xv = s_x[r_lo + row];
          const uint4 w = tile[(size_t)row * q.KV + cv];
          a8[0] = fmaf(__uint_as_float(w.x << 16), xv, a8[0]);
          a8[1] = fmaf(__uint_as_float(w.x & 0xFFFF0000u), xv, a8[1]);
          a8[2] = fmaf(__uint_as_float(w.y << 16), xv, a8[2]);
          a8[3] = fmaf(__uint_as_float(w.y & 0xFFFF0000u), xv, a8[3]);
          a8[4] = fmaf(__uint_as_float(w.z << 16), xv, a8[4]);
          a8[5] = fmaf(__uint_as_float(w.z & 0xFFFF0000u), xv, a8[5]);
          a8[6] = fmaf(__uint_as_float(w.w << 16), xv, a8[6]);
          a8[7] = fmaf(__uint_as_float(w.w & 0xFFFF0000u), xv, a8[7]);
        }
      }
#pragma unroll 1
      for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int e = 0; e < 8; ++e) a8[e] += __shfl_xor_sync(0xffffffffu, a8[e], o);
      }
      if (q.sub == 0) {
        float4* dst = reinterpret_cast<float4*>(s_red + warp * 512 + cv * 8);
        dst[0] = make_float4(a8[0], a8[1], a8[2], a8[3]);
        dst[1] = make_float4(a8[4], a8[5], a8[6], a8[7]);
      }
    }
    if (!ok && !*abort) fail(p, misc);
    tr.mark(3);
    csync();
    if (*abort) return false;
    if (prow > 0) {
#pragma unroll 1
      for (int j = tid; j < k; j += kNC) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kNW; ++w) sum += s_red[w * 512 + j];
        const long long v = scale != 0.0 ? __double2ll_rn((double)sum * scale) : 0ll;
        red_add_u64(acc + (size_t)j * kAccStride, (1ull << kCountShift) + (unsigned long long)v);
      }
    }
    tr.mark(4);

    // ---- C. exchange 1: wait until every contributing CTA has been added.  One
    //      thread watches one word (thousands of pollers on the accumulators
    //      would delay the very atomics they wait for); then every thread
    //      validates its own word, which is normally complete by then.
    if (tid == 0) {
      const unsigned long long* wp = acc + (size_t)(k - 1) * kAccStride;
      unsigned it = 0;
      for (;;) {
        const unsigned long long w = ld_relaxed_u64(wp);
        if ((unsigned)((w + (1ull << (kCountShift - 1))) >> kCountShift) == (unsigned)n_contrib) break;
        if (++it > kSpinLimit || ((it & 1023u) == 0 && *abort)) {
          if (!*abort) fail(p, misc);
          break;
        }
      }
    }
    csync();
    if (*abort) return false;
#pragma unroll 1
    for (int j = tid; j < k; j += kNC) {
      unsigned long long w = 0;
      unsigned it = 0;
      for (;;) {
        w = ld_relaxed_u64(acc + (size_t)j * kAccStride);
        const unsigned cnt = (unsigned)((w + (1ull << (kCountShift - 1))) >> kCountShift);
        if (cnt == (unsigned)n_contrib) break;
        if (++it > kSpinLimit || ((it & 1023u) == 0 && *abort)) {
          if (!*abort) fail(p, misc);
          break;
        }
      }
      const long long val = (long long)(w - ((unsigned long long)n_contrib << kCountShift));
      s_c[j] = (float)((double)val * inv_scale);
    }
    csync();
    if (*abort) return false;
    tr.mark(5);

    // ---- D. pass 2 (residual rows of the basis chunks, still in the ring) and
    //      the image rows: the same eight-rows-per-lane-group loop over both
    const int hold_log2 = q.lpr_log2 - 3;  // lanes per held row after reduce8
    // all image chunks of this group must have landed (they were prefetched)
    // (one chunk per lane, all waits in flight together; the warp then agrees)
    {
      bool mine_ok = true;
      if (lane < ochunks) {
        const unsigned seq = n_p0 + pchunks + lane;
        mine_ok = mbar_wait(&full[seq % kSlots], (seq / kSlots) & 1u, abort);
      }
      ok = __all_sync(0xffffffffu, ok && mine_ok);
    }
    tr.mark(7);
    float sr = 0.f;
    // ---- E (first half). exchange 2 is published as soon as the residual rows are done, by
    //      the warp that hands in the last partial, so that its latency runs under the image
    //      rows.  A word is the partial (non-negative, or NaN) with the parity of the launch
    //      in its sign bit: the arrays start as zeros, the first launch writes sign 1, and
    //      every launch rewrites every word, so a word of this launch cannot be mistaken for
    //      the previous one's and no fence is needed for the decision.  148 partials are
    //      five 128-byte lines that every CTA reads.
    // A pair shares the first group's slot array: word cta is this CTA's partial of its own
    // group, words G + u carry ||x||^2 of group u for the other half of the grid.
    auto deposit = [&]() {
      sr = warp_sum(sr);
      if (lane == 0) {
        volatile float* part = s_red;
        part[warp] = sr;
        __threadfence_block();
        if (atomicAdd(&misc->deposits, 1) == kNW - 1) {
          __threadfence_block();
          float t = 0.f;   // fixed order: the sum does not depend on who came last
#pragma unroll
          for (int w = 0; w < kNW; ++w) t += part[w];
          unsigned* slots = reinterpret_cast<unsigned*>(gA.slot_r);
          st_relaxed_u32(slots + cta, (__float_as_uint(t) & 0x7fffffffu) | (tag << 31));
          if (len == 2 && lc == 0)
            st_relaxed_u32(slots + G + (second ? 1 : 0),
                           (__float_as_uint(sum2) & 0x7fffffffu) | (tag << 31));
        }
      }
    };
    // work items: lane groups take eight rows at a time, first of the basis slab, then of
    // the image slab (rows per chunk are a multiple of 8, so an item stays inside a chunk);
    // only items with rows are enumerated, rounded up to a whole warp of lane groups
    const int itemsP = (prow + 7) >> 3, n_live = itemsP + ((orow + 7) >> 3);
    const int n_items = ((n_live + (1 << rpp_log2) - 1) >> rpp_log2) << rpp_log2;
    const int lanegroups = kNW << rpp_log2;          // lane groups in the CTA
    // The warps that hold basis items run them alone: the others hand in an empty partial
    // and start their image items only when the last basis item is done (named barrier 2:
    // they wait, the basis warps only arrive), so the partial is published as early as
    // possible.  Every warp takes part exactly once per phase, whatever `ok` says.
    const bool basis_warp = (warp << rpp_log2) < itemsP;
    bool deposited = !basis_warp;
    if (!basis_warp) {
      deposit();
      asm volatile("bar.sync 2, %0;" ::"n"(kNC) : "memory");
    }
    if (ok) {
      int released = 0;  // chunks this warp has already given back to the producer
#pragma unroll 1
      for (int item = (warp << rpp_log2) + q.sub; item < n_items; item += lanegroups) {
        const bool image = item >= itemsP;
        const int row0g = (image ? item - itemsP : item) << 3;   // first row, within the slab
        const int cj = row0g >> q.rc_log2;
        const int ci = min((image ? pchunks : 0) + cj, pchunks + ochunks - 1);
        // items come in chunk order: every chunk before this warp's current one is done
        // (n_items is a multiple of the lane groups per warp, so the warp stays converged)
        const int ci_warp = __shfl_sync(0xffffffffu, ci, 0);
        if (lane == 0)
          for (; released < ci_warp; ++released) mbar_arrive(&empty[(n_p0 + released) % kSlots]);
        released = ci_warp;
        const unsigned sl = (n_p0 + ci) % kSlots;
        const uint4* tile = reinterpret_cast<const uint4*>(ring + (size_t)sl * kChunk);
        const int r_lo = cj << q.rc_log2, rows = min(rc, (image ? orow : prow) - r_lo);
        const int row0 = row0g & (rc - 1);
        float v[8];
        dot8(tile, s_c, q, row0, rows, v);
        const float dot = reduce8(v, q.cl, LPR);
        const int row = row0 + (q.cl >> hold_log2);
        if ((q.cl & ((1 << hold_log2) - 1)) == 0 && row < rows) {
          if (image) {
            y_tok[s.o0 + r_lo + row] = nonfinite ? __int_as_float(0x7fc00000) : dot;
          } else {
            const float rv = s_x[r_lo + row] - dot;
            g.r[s.p0 + r_lo + row] = rv;
            sr = fmaf(rv, rv, sr);
          }
        }
        // basis items come first: once none is left for this warp, its partial is final
        if (!deposited && item - q.sub + lanegroups >= itemsP) {
          deposit();
          deposited = true;
          asm volatile("bar.arrive 2, %0;" ::"n"(kNC) : "memory");
        }
      }
      __syncwarp();
      if (lane == 0) {
#pragma unroll 1
        for (; released < pchunks + ochunks; ++released)
          mbar_arrive(&empty[(n_p0 + released) % kSlots]);
      }
    }
    if (!deposited) {   // only after a failed wait: keep the barrier count whole
      deposit();
      asm volatile("bar.arrive 2, %0;" ::"n"(kNC) : "memory");
    }
    tr.mark(8);
    if (!ok && !*abort) fail(p, misc);
    n += pchunks + ochunks;

    // ---- E (second half). exchange 2: collect, decide.
    if (warp == 0) {
      // one warp polls all words (lane l owns words l, l+32, ...); each word is
      // validated by the launch parity in its sign bit
      float vals[8];
      unsigned it = 0;
      bool done = false;
      while (!done) {
        bool all = true;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int t = lane + 32 * i;
          vals[i] = 0.f;
          if (t < G + (len == 2 ? 2 : 0)) {
            const unsigned w = ld_relaxed_u32(reinterpret_cast<const unsigned*>(gA.slot_r) + t);
            all = all && ((w >> 31) == (tag & 1u));
            vals[i] = __uint_as_float(w & 0x7fffffffu);
          }
        }
        done = __all_sync(0xffffffffu, all);
        if (!done && (++it > kSpinLimit || ((it & 1023u) == 0 && *abort))) {
          if (!*abort && lane == 0) fail(p, misc);
          break;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) s_vals[lane + 32 * i] = vals[i];
    }
    csync();
    tr.mark(10);
    if (*abort) return false;
    {  // every warp folds the slots of each group in the same fixed order
      const int split = gA.ncta;   // the whole grid when the group is alone
      float tA = 0.f, tB = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int t = lane + 32 * i;
        const float v = s_vals[t];
        tA += t < split ? v : 0.f;
        tB += (t >= split && t < G) ? v : 0.f;
      }
      tA = warp_sum(tA);
      if (len == 2) tB = warp_sum(tB);
      // ||r|| < eps ||x||  <=>  ||r||^2 < eps^2 ||x||^2  (both sides >= 0); NaN compares false
      const float t = second ? tB : tA;
      const double e2 = (double)g.eps * (double)g.eps;
      const bool fast = !nonfinite && ((double)t < e2 * (double)sum2);
      gate = fast ? 0 : 1;
      if (lc == 0 && tid == 0) {
        const size_t at = ((size_t)slot_io * p.log_step_stride + gi_mine) * p.n_tokens + p.token;
        p.gate_log[at] = (unsigned char)gate;
        if (p.rho_log)
          p.rho_log[at] = nonfinite ? __int_as_float(0x7fc00000) : sqrtf(__fdividef(t, sum2));
      }
      if (len == 2) {  // the partner's decision, from its partial sums and its ||x||^2
        const PersistGroup& go = second ? gA : gB;
        const float to = second ? tA : tB, s2o = s_vals[G + (second ? 0 : 1)];
        const double e2o = (double)go.eps * (double)go.eps;
        const bool finite_o = s2o - s2o == 0.f;
        const bool fast_o = finite_o && ((double)to < e2o * (double)s2o);
        gate_other = (!fast_o && finite_o && !(go.flags & GSI_FLAG_STATIC_PROJECTION)) ? 1 : 0;
      }
    }
    gate = gate && !(g.flags & GSI_FLAG_STATIC_PROJECTION) && !nonfinite;
    tr.mark(11);
  } else {
    if (zeroer && tid < 3) g.bar[2 * tid + (parity ^ 1u)] = 0u;
    if (cta == 0 && tid == 0)
      p.gate_log[((size_t)slot_io * p.log_step_stride + gi) * p.n_tokens + p.token] = 1;
    if (tid < next_len * kDescWords) *desc_dst = desc_word;
    csync();
    if (has_next) prefetch_next_x(g_next, slot_io, p.n_tokens);
    if (next_len == 2) prefetch_next_x(desc(gi + len + 1), slot_io, p.n_tokens, 1);
  }

  // ---- F. gated residual of every gated group of the phase, each with the whole grid
#pragma unroll 1
  for (int u = 0; u < len; ++u) {
    const PersistGroup& gg = u ? gB : gA;
    const int fire = ((u == 1) == second) ? gate : gate_other;
    if (!fire) continue;
    if (!dense) {
      // r (and the image rows of y) were written by other CTAs: make them visible grid-wide
      // before anyone reads them (release fence, arrival count, acquire fence).  Only gated
      // groups pay for this.
      if (tid == 0) {
        __threadfence();
        grid_arrive_wait(gg.bar + 2 + parity, (unsigned)G, p, misc);
        __threadfence();
      }
      csync();
      if (*abort) return false;
    }
    Slab sw;
    sw.p0 = sw.p1 = 0;
    sw.o0 = min(gg.O, cta * gg.o_rows_w);
    sw.o1 = min(gg.O, sw.o0 + gg.o_rows_w);
    gated_pass(gg, sw, dense ? rsrc : gg.r, gg.y + (size_t)p.token * gg.O, dense, smem);
    csync();
    tr.mark(12);
    // A dense group has no exchange: a grid barrier keeps the groups of a dense stack in
    // model order.  After a gated residual none is needed: no CTA passes exchange 1 of the
    // next phase before every CTA has posted its partial there, which it does after this.
    if (dense) {
      if (tid == 0) grid_arrive_wait(gg.bar + parity, (unsigned)G, p, misc);
      csync();
      tr.mark(13);
      if (*abort) return false;
    }
  }
  return true;
}

template <bool kPairs, int kK>
__device__ void consumer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  Ctx ctx;
  ctx.step = p.use_counter ? *p.step : 0;
  ctx.slot_io = ctx.step % p.n_steps;
  const int epoch = *p.epoch;
  ctx.parity = (unsigned)epoch & 1u;
  ctx.tag = (unsigned)epoch + 1u;
  ctx.n = 0;
  ctx.tr.start(p);
  // the first phase's descriptors (the second slot is used only if the phase is a pair)
  if ((int)threadIdx.x < min(p.n_groups, 2) * kDescWords) {
    const int j = threadIdx.x >= kDescWords ? 1 : 0;
    reinterpret_cast<uint32_t*>(smem + kOffDesc + j * 512)[threadIdx.x - j * kDescWords] =
        __ldg(reinterpret_cast<const uint32_t*>(p.groups) + threadIdx.x);
  }
  csync();
  bool ok = true;
  ctx.len = 1;
#pragma unroll 1
  for (int gi = 0; gi < p.n_groups && ok; gi += ctx.len) ok = group_phase<kPairs, kK>(p, smem, misc, ctx, gi);
  // Every CTA read the counters at its start and has since taken part in the
  // last group's exchange, so they may advance now.
  if (blockIdx.x == 0 && threadIdx.x == 0 && ok) {
    *p.epoch = epoch + 1;
    if (p.use_counter && p.advance) *p.step = ctx.step + 1;
  }
}

template <bool kPairs, int kK>
__global__ void __launch_bounds__(kThreadsP, 1) k_decode_step(PersistParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kSlots;
  Misc* misc = reinterpret_cast<Misc*>(smem + kOffMisc);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kNW);
    }
    misc->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x >= kNC) {
    if (threadIdx.x == kNC) producer(p, smem, misc);
    return;
  }
  consumer<kPairs, kK>(p, smem, misc);
}

template <bool kPairs, int kK>
cudaError_t launch_decode_step_t(const PersistParams& p, int grid, cudaStream_t st) {
  static bool configured[64] = {};   // per device: the attribute belongs to the device's function
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_step<kPairs, kK>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  PersistParams pp = p;
  void* args[] = {&pp};
  // cooperative launch: all CTAs are guaranteed co-resident, which the
  // cross-CTA exchanges rely on
  cudaError_t e = cudaLaunchCooperativeKernel((void*)k_decode_step<kPairs, kK>, dim3(grid),
                                              dim3(kThreadsP), args, kSmemBytes, st);
  if (e != cudaSuccess && getenv("GSI_VERBOSE"))
    fprintf(stderr, "gsi: persistent launch failed: %s\n", cudaGetErrorString(e));
  return e;
}

}  // namespace

}  // namespace gsi
