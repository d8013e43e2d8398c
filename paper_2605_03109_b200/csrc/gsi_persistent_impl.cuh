// Persistent decode-step kernel: every group of the stack in ONE launch.
//
// One CTA per SM.  Each CTA owns a fixed slab of rows of every basis P and of every
// (concatenated) image W_P, and a fixed set of rows of every weight matrix W.  A producer
// warp streams ALL weights from HBM into a ring of shared-memory slots: the slabs of P and
// W_P with bulk async copies, the rows of W (gated residual, dense baseline) as TMA boxes of
// up to 30 rows x 256 columns.  Weight addresses never depend on x, so the next group's slabs
// arrive while the current group waits on its exchange.  Fifteen consumer warps run
// Algorithm 1 per group (two consecutive groups declared independent share a phase on two
// parts of the grid).  A phase has ONE grid-wide exchange:
//
//   statistics  warp 0: max |x| and sum x^2 over this CTA's rows of x; the maximum is
//               published as a tagged 32-bit word (no fence: the word validates itself)
//   pass 1      partial c = P_slab^T x_slab                              (line 1)
//   exchange    every CTA adds, as 64-bit fixed-point numbers whose upper bits count the
//               arrivals (integer addition is order-free, so the sums are bit-reproducible):
//               its partial c_j (scale from the global max |x|, collected from the tagged
//               words meanwhile), its partial ||x||^2, and its partial ||r||^2 of the
//               PREVIOUS phase; it then polls the words until all have arrived
//   gate        of the previous phase, from the exact integer sums: the same decision on
//               every CTA                                                (line 4, Eq. (3.3))
//   pass 2      r_slab = x_slab - P_slab c, partial ||r||^2              (lines 2-3)
//   gated       y_rows += W_rows r of the groups of the phase before the previous one
//               whose gate fired (their boxes follow this phase's basis slab in the ring;
//               r and the image rows were made visible by a fenced arrival counter that
//               every CTA posted when the gate was decided)              (Eq. (3.2))
//   image       y_rows = W_P,rows c                                      (line 5)
//
// so the gate of a phase is known one exchange later and its residual runs one phase after
// that: every group's inputs are pre-staged buffers (the contract of the stack driver), and
// all of y is complete when the launch ends.  Two ticks after the last phase settle the
// remaining gates and residuals.
//
// Every wait is bounded; a wait that gives up records GSI_ERR_TIMEOUT in the status word,
// the CTA drains its copies in flight and returns.
//
// This header holds the kernel; every build of it (with or without the pair logic, for any
// rank or for one rank) is compiled in a translation unit of its own.
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
constexpr int kBoxCols = kPersistBoxCols;
constexpr unsigned kLocalSpinLimit = 1u << 24;   // waits inside the CTA (ring, producer hand-off)
constexpr int kCountShift = 54;
constexpr unsigned long long kOne = 1ull << kCountShift;

// shared memory map (bytes)
constexpr int kOffBar = 0;          // full[kSlots], empty[kSlots]
constexpr int kOffMisc = 256;       // scalars
constexpr int kOffX = 512;          // x of this CTA's basis rows, two buffers (kPersistMaxPRows floats each)
constexpr int kOffC = kOffX + 2 * kPersistMaxPRows * 4;   // c (512 floats)
constexpr int kOffDesc = kOffC + 2048;                    // 4 group descriptors, 512 B each
constexpr int kDescSlots = 4;
constexpr int kOffRed = kOffDesc + kDescSlots * 512;      // cross-warp scratch (kNW*512 floats)
constexpr int kOffRs = kOffRed + kNW * 512 * 4;           // staged slice of r (16 KB)
constexpr int kOffYacc = kOffRs + kSlice * 4;             // per-row accumulators (kPersistMaxORows floats)
constexpr int kOffRing = ((kOffYacc + kPersistMaxORows * 4 + 1023) / 1024) * 1024;
constexpr int kSmemBytes = kOffRing + kSlots * kChunk;
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 CTA");
static_assert(sizeof(PersistGroup) <= 512 && sizeof(PersistGroup) % 4 == 0, "descriptor slot");
static_assert(kPersistBoxRowsMax * kBoxCols * 2 <= kChunk, "a box fits a slot");
static_assert(kPersistBoxRowsMax == 2 * kNW, "two rows of a box per consumer warp");
constexpr int kDescWords = (int)(sizeof(PersistGroup) / 4);

struct Misc {
  int abort;
  unsigned amax_bits;       // max |x| of this phase's group (>= 0x7f800000: a non-finite token)
  float x2_part;            // this CTA's sum of x^2 over its rows
  double x2;                // ||x||^2 of this phase's group
  int fire[4];              // decisions on the previous phase's groups, by tick parity: 1 = stream W
  float sr[kNW];            // per-warp partial ||r||^2 of this phase
  volatile unsigned decision[4];   // hand-off to the producer: (phase + 1) << 8 | fire mask
};
static_assert(sizeof(Misc) <= 256, "scalars");

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
  for (unsigned it = 0; it < kLocalSpinLimit; ++it) {
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
// One box of a 2-D tensor map (no multicast): x = first column, y = first row.
__device__ __forceinline__ void tma_box_g2s(void* dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void cp_async4(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
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

__device__ __forceinline__ void fail(const PersistParams& p, Misc* misc) {
  misc->abort = 1;
  atomicExch(p.status, (int)GSI_ERR_TIMEOUT);
}

// Optional cycle trace (thread 0 of every CTA; sections of the per-phase pipeline, summed
// over phases); p.trace == nullptr disables it.
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
  int o0, o1;  // rows of the concatenated images owned by this CTA
};
__device__ __forceinline__ Slab slab_of(const PersistGroup& g, int lc) {
  Slab s;
  s.p0 = min(g.d, lc * g.p_rows);
  s.p1 = min(g.d, s.p0 + g.p_rows);
  s.o0 = min(g.O, lc * g.o_rows);
  s.o1 = min(g.O, s.o0 + g.o_rows);
  return s;
}

// ------------------------------------------------------------------ producer
struct Ring {
  uint64_t* full;
  uint64_t* empty;
  unsigned char* slots;
  unsigned n;   // sequence number of the next chunk
};

// Wait for the slot of chunk n to be free; false = give up.
__device__ __forceinline__ bool ring_acquire(Ring& rg, volatile int* abort) {
  const unsigned slot = rg.n % kSlots, ph = (rg.n / kSlots) & 1u;
  return mbar_wait(&rg.empty[slot], ph ^ 1u, abort);
}

// The W boxes of one group for this CTA, in the order the consumers take them: column
// slices of 4096 outermost (one staged slice of r serves them), then maps, then row blocks,
// then the 256-column boxes of the slice.
__device__ bool produce_w(const PersistGroup& g, Ring& rg, volatile int* abort) {
  const int cta = blockIdx.x;
  const int nsl = (g.d + kSlice - 1) / kSlice;
  for (int sl = 0; sl < nsl; ++sl) {
    const int c0 = sl * kSlice, ncb = (min(kSlice, g.d - c0) + kBoxCols - 1) / kBoxCols;
    for (int j = 0; j < g.n_maps; ++j) {
      const int dout = g.off[j + 1] - g.off[j], rows = g.w_rows[j], rb = g.w_rb[j];
      const int row0 = cta * rows;
      const int live = min(rows, dout - row0);
      const char* tm = static_cast<const char*>(g.tmW) + (size_t)j * kPersistTmapBytes;
      for (int b = 0; b * rb < live; ++b) {
        for (int cb = 0; cb < ncb; ++cb) {
          if (!ring_acquire(rg, abort)) return false;
          const unsigned slot = rg.n % kSlots;
          mbar_expect_tx(&rg.full[slot], (uint32_t)rb * kBoxCols * 2);
          tma_box_g2s(rg.slots + (size_t)slot * kChunk, tm, c0 + cb * kBoxCols, row0 + b * rb,
                      &rg.full[slot]);
          ++rg.n;
        }
      }
    }
  }
  return true;
}

// Rows [a, b) of a row-major [rows][k] bf16 matrix as chunks of whole rows.
__device__ bool produce_rows(const uint16_t* base, int k, int a, int b, Ring& rg, volatile int* abort) {
  const int rc = kChunk / (k * 2);
  for (int r = a; r < b; r += rc) {
    const int rows = min(rc, b - r);
    if (!ring_acquire(rg, abort)) return false;
    const unsigned slot = rg.n % kSlots;
    const uint32_t bytes = (uint32_t)rows * k * 2;
    mbar_expect_tx(&rg.full[slot], bytes);
    bulk_g2s(rg.slots + (size_t)slot * kChunk, base + (size_t)r * k, bytes, &rg.full[slot]);
    ++rg.n;
  }
  return true;
}

__device__ void producer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  Ring rg;
  rg.full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  rg.empty = rg.full + kSlots;
  rg.slots = smem + kOffRing;
  rg.n = 0;
  volatile int* abort = &misc->abort;
  const int cta = blockIdx.x;
  bool ok = true;
  // ticks: tick t runs phase t (while there is one) and the gated residuals of phase t - 2
  int gi = 0;        // first group of phase t
  int g_pp = -1, len_pp = 0;   // phase t - 2
  int g_p = -1, len_p = 0;     // phase t - 1
  for (int t = 0; ok; ++t) {
    const bool own = gi < p.n_groups;
    if (!own && len_p == 0 && len_pp == 0) break;
    int len = 0;
    const PersistGroup* g = nullptr;
    if (own) {
      const PersistGroup& gA = p.groups[gi];
      len = gA.phase_len;
      g = (len == 2 && cta >= gA.cta0 + gA.ncta) ? &p.groups[gi + 1] : &gA;
    }
    const bool dense = own && (g->flags & GSI_FLAG_DENSE);
    Slab s{};
    if (own && !dense) {
      s = slab_of(*g, cta - g->cta0);
      ok = produce_rows(g->P, g->k, s.p0, s.p1, rg, abort);
    }
    if (ok && len_pp > 0) {
      // the decision on phase t - 2 (taken by the consumers during tick t - 1)
      const unsigned want = (unsigned)(t - 1);   // (phase + 1)
      unsigned v = 0, it = 0;
      for (;;) {
        v = misc->decision[(t - 2) & 3];
        if ((v >> 8) == want) break;
        if (++it > kLocalSpinLimit || *abort) {
          ok = false;
          break;
        }
      }
      for (int u = 0; ok && u < len_pp; ++u)
        if (v & (1u << u)) ok = produce_w(p.groups[g_pp + u], rg, abort);
    }
    if (ok && own) {
      if (dense)
        ok = produce_w(*g, rg, abort);
      else
        ok = produce_rows(g->WP, g->k, s.o0, s.o1, rg, abort);
    }
    g_pp = g_p;
    len_pp = len_p;
    g_p = gi;
    len_p = len;
    gi += len;
  }
  if (!ok && !*abort) fail(p, misc);
  // Every copy issued must have landed before the CTA may give up its shared
  // memory: wait (bounded) for the last kSlots chunks.
  {
    const unsigned first = rg.n > (unsigned)kSlots ? rg.n - kSlots : 0;
    for (unsigned c = first; c < rg.n; ++c) {
      const unsigned slot = c % kSlots, ph = (c / kSlots) & 1u;
      for (unsigned it = 0; it < kLocalSpinLimit; ++it)
        if (mbar_try(&rg.full[slot], ph)) break;
    }
  }
}

// ------------------------------------------------------------------ consumer
// Lane layout over a row of k bf16: KV = k/8 vectors, LPR = min(32, KV) lanes
// per row, RPP = 32/LPR rows per warp pass, VPL = KV/LPR vectors per lane.

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
// Smallest e with v < 2^e for a positive finite double v (binary exponent + 1).
__device__ __forceinline__ int exp_above(double v) {
  return ((__double2hiint(v) >> 20) & 0x7ff) - 1022;
}

// Grid-wide arrival counter: wait (bounded) until `target` arrivals have been added.
__device__ __forceinline__ bool grid_wait(const unsigned* ctr, unsigned target, const PersistParams& p,
                                          Misc* misc) {
  volatile int* abort = &misc->abort;
  unsigned it = 0;
  while (ld_relaxed_u32(ctr) < target) {
    if (++it > p.spin_limit || *abort) {
      if (!*abort) fail(p, misc);
      return false;
    }
  }
  return true;
}

// Poll one accumulator until `n` arrivals have been added; returns the signed sum.
__device__ __forceinline__ long long poll_acc(const unsigned long long* wp, unsigned n,
                                              const PersistParams& p, Misc* misc) {
  volatile int* abort = &misc->abort;
  unsigned long long w = 0;
  unsigned it = 0;
  for (;;) {
    w = ld_relaxed_u64(wp);
    if ((unsigned)((w + (kOne >> 1)) >> kCountShift) == n) break;
    if (++it > p.spin_limit || ((it & 1023u) == 0 && *abort)) {
      if (!*abort) fail(p, misc);
      break;
    }
  }
  return (long long)(w - ((unsigned long long)n << kCountShift));
}

struct Ctx {
  int slot_io;
  unsigned parity, tag;
  Ring rg;        // consumer's view: n advances exactly as in producer()
  Trace tr;
};

// ---- W stream: y_rows (+)= W_rows . src (src = r of a gated group, or x for the dense
// baseline), boxes taken from the ring in the producer's order.  Out of line: most phases
// skip it.  Returns false when a wait gave up.
__device__ __noinline__ bool w_stream(const PersistParams& p, const PersistGroup& g, const float* src,
                                      float* y, bool dense, unsigned char* smem, Ctx& ctx,
                                      Misc* misc) {
  float* s_rs = reinterpret_cast<float*>(smem + kOffRs);
  float* s_yacc = reinterpret_cast<float*>(smem + kOffYacc);
  volatile int* abort = &misc->abort;
  Ring& rg = ctx.rg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cta = blockIdx.x;
  const int nsl = (g.d + kSlice - 1) / kSlice;
  bool ok = true;
#pragma unroll 1
  for (int sl = 0; sl < nsl; ++sl) {
    const int c0 = sl * kSlice, cols = min(kSlice, g.d - c0);
    const int ncb = (cols + kBoxCols - 1) / kBoxCols;
    csync();
    // Stage the slice so that a lane's two 16-byte loads per box are conflict-free: within a
    // 256-column block, the first halves of the 32 lanes' eight columns, then the second halves.
#pragma unroll 1
    for (int i = tid; i < ncb * 64; i += kNC) {
      const int col = i * 4;
      const float4 v = col < cols ? __ldcg(reinterpret_cast<const float4*>(src + c0 + col))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
      const int blk = i >> 6, w4 = i & 63;
      reinterpret_cast<float4*>(s_rs)[blk * 64 + (w4 & 1) * 32 + (w4 >> 1)] = v;
    }
    csync();
    int ybase = 0;
#pragma unroll 1
    for (int j = 0; j < g.n_maps; ++j) {
      const int dout = g.off[j + 1] - g.off[j], rows = g.w_rows[j], rb = g.w_rb[j];
      const int live = min(rows, dout - cta * rows);
      const bool mine = 2 * warp < rb;
#pragma unroll 1
      for (int b = 0; b * rb < live; ++b) {
        unsigned long long a0 = 0ull, a1 = 0ull;
#pragma unroll 1
        for (int cb = 0; cb < ncb; ++cb) {
          const unsigned slot = rg.n % kSlots, ph = (rg.n / kSlots) & 1u;
          ++rg.n;
          if (ok && !mbar_wait(&rg.full[slot], ph, abort)) ok = false;
          if (ok && mine) {
            const uint4* tile = reinterpret_cast<const uint4*>(rg.slots + (size_t)slot * kChunk);
            const uint4 w0 = tile[(2 * warp) * (kBoxCols / 8) + lane];
            const uint4 w1 = tile[(2 * warp + 1) * (kBoxCols / 8) + lane];
            const float4 ra = reinterpret_cast<const float4*>(s_rs)[cb * 64 + lane];
            const float4 rb4 = reinterpret_cast<const float4*>(s_rs)[cb * 64 + 32 + lane];
            const unsigned long long r0 = pack2(ra.x, ra.y), r1 = pack2(ra.z, ra.w);
            const unsigned long long r2 = pack2(rb4.x, rb4.y), r3 = pack2(rb4.z, rb4.w);
            fma2(a0, bf16x2_to_f32x2(w0.x), r0);
            fma2(a1, bf16x2_to_f32x2(w1.x), r0);
            fma2(a0, bf16x2_to_f32x2(w0.y), r1);
            fma2(a1, bf16x2_to_f32x2(w1.y), r1);
            fma2(a0, bf16x2_to_f32x2(w0.z), r2);
            fma2(a1, bf16x2_to_f32x2(w1.z), r2);
            fma2(a0, bf16x2_to_f32x2(w0.w), r3);
            fma2(a1, bf16x2_to_f32x2(w1.w), r3);
          }
          __syncwarp();
          if (ok && lane == 0) mbar_arrive(&rg.empty[slot]);
        }
        if (mine) {
          const float t0 = warp_sum(sum2(a0)), t1 = warp_sum(sum2(a1));
          if (lane == 0) {
            const int i0 = ybase + b * rb + 2 * warp;
            s_yacc[i0] = (sl == 0 ? 0.f : s_yacc[i0]) + t0;
            s_yacc[i0 + 1] = (sl == 0 ? 0.f : s_yacc[i0 + 1]) + t1;
          }
        }
      }
      ybase += ((live > 0 ? (live + rb - 1) / rb : 0)) * rb;
    }
  }
  if (!ok && !*abort) fail(p, misc);
  csync();
  // rows back to y: the same walk over the maps
  {
    int ybase = 0;
#pragma unroll 1
    for (int j = 0; j < g.n_maps; ++j) {
      const int dout = g.off[j + 1] - g.off[j], rows = g.w_rows[j], rb = g.w_rb[j];
      const int live = min(rows, dout - cta * rows);
      if (ok) {
#pragma unroll 1
        for (int i = tid; i < live; i += kNC) {
          float* yp = y + g.off[j] + cta * rows + i;
          *yp = dense ? s_yacc[ybase + i] : (__ldcg(yp) + s_yacc[ybase + i]);
        }
      }
      ybase += ((live > 0 ? (live + rb - 1) / rb : 0)) * rb;
    }
  }
  return ok;
}


// Items of eight rows (one lane group each) over the rows of `nchunks` ring chunks that start
// at sequence number n0.  Item ids [id0, id0 + n_ids) of the phase's joint numbering belong to
// this part; ids are dealt round-robin to the lane groups of the CTA, so the basis rows and the
// image rows of a phase load the warps evenly.  kImage: out[row] = dot (NaN for a non-finite
// token); otherwise out[row] = x[row] - dot and the return value is this lane's share of
// ||r||^2.  Every warp gives every chunk back exactly once.
template <bool kImage>
__device__ __forceinline__ float row_items(const Geo& q, Ring& rg, unsigned n0, int nchunks, int nrows,
                                           int id0, int n_ids, const float* s_c, const float* s_x,
                                           float* out, bool nonfinite, bool ok) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int LPR = 1 << q.lpr_log2, rpp_log2 = 5 - q.lpr_log2, rc = 1 << q.rc_log2;
  const int hold_log2 = q.lpr_log2 - 3;          // lanes per held row after reduce8
  const int lanegroups = kNW << rpp_log2;
  float sr = 0.f;
  int released = 0;
  if (ok) {
    int id = (warp << rpp_log2) + q.sub;
    if (id < id0) id += ((id0 - id + lanegroups - 1) / lanegroups) * lanegroups;
#pragma unroll 1
    for (; id < id0 + n_ids; id += lanegroups) {
      const int row0g = (id - id0) << 3;                       // first row, within the slab
      const int ci = min(row0g >> q.rc_log2, nchunks - 1);
      const int ci_warp = __shfl_sync(0xffffffffu, ci, 0);     // ids ascend with the lane
      if (lane == 0)
        for (; released < ci_warp; ++released) mbar_arrive(&rg.empty[(n0 + released) % kSlots]);
      released = ci_warp;
      const uint4* tile =
          reinterpret_cast<const uint4*>(rg.slots + (size_t)((n0 + ci) % kSlots) * kChunk);
      const int r_lo = ci << q.rc_log2, rows = min(rc, nrows - r_lo);
      const int row0 = row0g - r_lo;
      float v[8];
      dot8(tile, s_c, q, row0, rows, v);
      const float dot = reduce8(v, q.cl, LPR);
      const int row = row0 + (q.cl >> hold_log2);
      if ((q.cl & ((1 << hold_log2) - 1)) == 0 && row < rows && row0g < nrows) {
        if (kImage) {
          out[r_lo + row] = nonfinite ? __int_as_float(0x7fc00000) : dot;
        } else {
          const float rv = s_x[r_lo + row] - dot;
          out[r_lo + row] = rv;
          sr = fmaf(rv, rv, sr);
        }
      }
    }
    __syncwarp();
    if (lane == 0)
      for (; released < nchunks; ++released) mbar_arrive(&rg.empty[(n0 + released) % kSlots]);
  }
  return sr;
}

// All chunks [n0, n0 + count) have landed (one chunk per lane, all waits in flight together).
__device__ __forceinline__ bool chunks_landed(Ring& rg, unsigned n0, int count, volatile int* abort) {
  const int lane = threadIdx.x & 31;
  bool mine_ok = true;
  for (int c = lane; c < count; c += 32) {
    const unsigned seq = n0 + c;
    mine_ok = mine_ok && mbar_wait(&rg.full[seq % kSlots], (seq / kSlots) & 1u, abort);
  }
  return __all_sync(0xffffffffu, mine_ok);
}

// kPairs = false compiles the pair logic out: stacks without concurrent groups run a smaller
// loop (the per-phase code has to stay resident in the instruction cache).  kK != 0 is a
// build for stacks whose groups all have rank kK (shifts, strides and loop bounds become
// constants); kK = 0 reads the rank from the descriptor.
template <bool kPairs, int kK>
__device__ void consumer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  float* s_xb = reinterpret_cast<float*>(smem + kOffX);
  float* s_c = reinterpret_cast<float*>(smem + kOffC);
  float* s_red = reinterpret_cast<float*>(smem + kOffRed);
  volatile int* abort = &misc->abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;

  Ctx ctx;
  ctx.rg.full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  ctx.rg.empty = ctx.rg.full + kSlots;
  ctx.rg.slots = smem + kOffRing;
  ctx.rg.n = 0;
  Ring& rg = ctx.rg;
  const int step = p.use_counter ? *p.step : 0;
  const int slot_io = step % p.n_steps;
  ctx.slot_io = slot_io;
  const int epoch = *p.epoch;
  const unsigned parity = (unsigned)epoch & 1u, tag = ((unsigned)epoch + 1u) & 1u;
  ctx.parity = parity;
  ctx.tag = tag;
  Trace& tr = ctx.tr;
  tr.start(p);

  auto desc = [&](int i) -> const PersistGroup& {
    return *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (i & (kDescSlots - 1)) * 512);
  };
  // the group of phase [i, i + len) whose fast path this CTA runs
  auto mine_of = [&](int i, int len) -> int {
    if (!kPairs || len < 2) return i;
    const PersistGroup& a = desc(i);
    return cta >= a.cta0 + a.ncta ? i + 1 : i;
  };
  // warp 0: request this CTA's rows of x of group gn into buffer `buf`
  auto request_x = [&](const PersistGroup& gn, int buf) {
    if (gn.flags & GSI_FLAG_DENSE) return;
    const Slab sn = slab_of(gn, cta - gn.cta0);
    const float* src = gn.x + (long long)slot_io * gn.x_step_stride + (size_t)p.token * gn.d + sn.p0;
    float* dst = s_xb + buf * kPersistMaxPRows;
    for (int i = lane; i < sn.p1 - sn.p0; i += 32) cp_async4(dst + i, src + i);
  };

  // the first phase's descriptors (the second slot is used only if the phase is a pair)
  if (tid < min(p.n_groups, 2) * kDescWords) {
    const int j = tid >= kDescWords ? 1 : 0;
    reinterpret_cast<uint32_t*>(smem + kOffDesc + j * 512)[tid - j * kDescWords] =
        __ldg(reinterpret_cast<const uint32_t*>(p.groups) + tid);
  }
  if (tid == 0) {
    misc->fire[0] = misc->fire[1] = misc->fire[2] = misc->fire[3] = 0;
    misc->decision[0] = misc->decision[1] = misc->decision[2] = misc->decision[3] = 0u;
  }
  csync();
  if (warp == 0) {
    const int len0 = kPairs ? desc(0).phase_len : 1;
    request_x(desc(mine_of(0, len0)), 0);
    cp_async_commit();
  }

  int gi = 0;
  int g_p = -1, len_p = 0;       // previous phase: its gates are settled in this tick
  int g_pp = -1, len_pp = 0;     // the phase before: its gated residuals run in this tick
  unsigned mask_pp = 0;
  bool contrib_p = false;        // this CTA holds a partial ||r||^2 of the previous phase
  int e_p = 0;                   // ... scaled by 2^(44 - e_p)
  unsigned long long* r2word_p = nullptr;
  bool ok = true;

#pragma unroll 1
  for (int t = 0; ok; ++t) {
    const bool own = gi < p.n_groups;
    if (!own && len_p == 0 && len_pp == 0) break;
    int len = 0, next_len = 0, gi_mine = gi;
    if (own) {
      const PersistGroup& gA = desc(gi);
      len = kPairs ? gA.phase_len : 1;
      next_len = kPairs ? gA.next_len : min(gA.next_len, 1);
      gi_mine = mine_of(gi, len);
    }
    const PersistGroup& g = desc(gi_mine);        // read only when `own`
    const bool dense = own && (g.flags & GSI_FLAG_DENSE);
    const bool gsi = own && !dense;
    const int lc = own ? cta - g.cta0 : 0;
    const int k = gsi ? (kK ? kK : g.k) : 0;
    Slab s{};
    if (gsi) s = slab_of(g, lc);
    const int prow = s.p1 - s.p0, orow = s.o1 - s.o0;
    float* s_x = s_xb + (t & 1) * kPersistMaxPRows;
    unsigned long long* acc = gsi ? g.acc + (size_t)parity * (k + 2) * kAccStride : nullptr;
    const int n_contrib = gsi ? (g.d + g.p_rows - 1) / g.p_rows : 0;

    Geo q{};
    if (gsi) {
      q.KV = k >> 3;
      q.lpr_log2 = q.KV >= 32 ? 5 : 31 - __clz(q.KV);
      q.vpl = q.KV > 32 ? q.KV >> 5 : 1;
      q.rc_log2 = 31 - __clz(kChunk / 2) - (31 - __clz(k));  // rows per chunk = 8192 / k
      q.sub = lane >> q.lpr_log2;
      q.cl = lane & ((1 << q.lpr_log2) - 1);
    }
    const int LPR = 1 << q.lpr_log2, rpp_log2 = 5 - q.lpr_log2, rc = 1 << q.rc_log2;
    const int pchunks = gsi ? (prow + rc - 1) >> q.rc_log2 : 0;
    const int ochunks = gsi ? (orow + rc - 1) >> q.rc_log2 : 0;

    // one word of the next phase's descriptors, in flight during the statistics
    uint32_t desc_word = 0;
    if (own && tid < next_len * kDescWords)
      desc_word = __ldg(reinterpret_cast<const uint32_t*>(p.groups + gi + len) + tid);

    // ---- A. statistics of this CTA's rows of x (warp 0), published at once
    if (gsi && warp == 0) {
      cp_async_wait_all();
      __syncwarp();
      float amax = 0.f, s2 = 0.f;
#pragma unroll 1
      for (int i = lane; i < prow; i += 32) {
        const float v = s_x[i];
        amax = fmaxf(amax, fabsf(v));
        s2 = fmaf(v, v, s2);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
      }
      // fmaxf drops NaN, the sum keeps it (and overflows to inf for huge inputs):
      // s2 - s2 is non-zero exactly when some x_i is NaN or inf (or x^2 overflowed)
      if (lane == 0) {
        const unsigned bits = (s2 - s2 == 0.f) ? __float_as_uint(amax) : 0x7fc00000u;
        if (prow > 0) st_relaxed_u32(g.xmax + lc, bits | (tag << 31));
        misc->x2_part = s2;
      }
    }
    if (own && tid < next_len * kDescWords) {
      uint32_t* dst = reinterpret_cast<uint32_t*>(
                          smem + kOffDesc +
                          ((gi + len + (tid >= kDescWords ? 1 : 0)) & (kDescSlots - 1)) * 512) +
                      (tid >= kDescWords ? tid - kDescWords : tid);
      *dst = desc_word;
    }
    if (tid == 0) misc->fire[(t & 1) * 2] = misc->fire[(t & 1) * 2 + 1] = 0;
    if (own && lc == gi_mine % g.ncta) {  // this CTA clears the group's counters for the next launch
      if (gsi) {
#pragma unroll 1
        for (int j = tid; j < k + 2; j += kNC)
          g.acc[((size_t)(parity ^ 1u) * (k + 2) + j) * kAccStride] = 0ull;
      }
      if (tid < 2) g.bar[2 * tid + (parity ^ 1u)] = 0u;
    }
    csync();
    tr.mark(0);
    if (warp == 0 && next_len > 0) {   // the next phase's rows of x travel while this phase runs
      request_x(desc(mine_of(gi + len, next_len)), (t + 1) & 1);
      cp_async_commit();
    }

    // ---- B. pass 1: partial c over this CTA's basis rows
    const unsigned n_p0 = rg.n;
    if (gsi) {
      ok = chunks_landed(rg, n_p0, pchunks, abort);
      tr.mark(1);
#pragma unroll 1
      for (int u = 0; u < q.vpl; ++u) {
        const int cv = q.cl + u * LPR;
        float a8[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a8[e] = 0.f;
#pragma unroll 1
        for (int ci = 0; ci < pchunks; ++ci) {
          if (!ok) break;
          const uint4* tile =
              reinterpret_cast<const uint4*>(rg.slots + (size_t)((n_p0 + ci) % kSlots) * kChunk);
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
      tr.mark(2);
      // ---- C. the group's max |x|: warp 0 collects the tagged words (lane l owns words
      //      l, l+32, ...), published about one pass earlier
      if (warp == 0) {
        unsigned m = 0, it = 0;
        bool done = false;
        while (!done) {
          bool all = true;
          m = 0;
#pragma unroll
          for (int i = 0; i < kPersistMaxGrid / 32; ++i) {
            const int w_i = lane + 32 * i;
            if (w_i < n_contrib) {
              const unsigned w = ld_relaxed_u32(g.xmax + w_i);
              all = all && ((w >> 31) == tag);
              m = max(m, w & 0x7fffffffu);
            }
          }
          done = __all_sync(0xffffffffu, all);
          if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
            if (!*abort && lane == 0) fail(p, misc);
            break;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) misc->amax_bits = m;
      }
    }
    csync();
    tr.mark(3);
    if (*abort) return;

    // ---- D. the exchange: this phase's partial c and ||x||^2, the previous phase's ||r||^2
    bool nonfinite = false;
    double inv_scale = 0.0;
    if (gsi) {
      const unsigned amax_bits = misc->amax_bits;
      nonfinite = amax_bits >= 0x7f800000u;
      const float amax = __uint_as_float(amax_bits);
      // fixed-point scales: |partial c_j| <= amax * rows * max|P| < 2^e, partial ||x||^2 <= rows * amax^2 < 2^ex
      double scale = 0.0, scale_x2 = 0.0;
      const float bound = amax * (float)g.p_rows * g.pmax;
      if (!nonfinite && bound > 0.f && bound < 3.0e38f) {
        const int e = max((int)((__float_as_uint(bound) >> 23) & 0xFFu), 1) - 126;
        scale = pow2d(43 - e);
        inv_scale = pow2d(e - 43);
        scale_x2 = pow2d(43 - exp_above((double)amax * (double)amax * (double)g.p_rows));
      }
      if (prow > 0) {
#pragma unroll 1
        for (int j = tid; j < k; j += kNC) {
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < kNW; ++w) sum += s_red[w * 512 + j];
          const long long v = scale != 0.0 ? __double2ll_rn((double)sum * scale) : 0ll;
          red_add_u64(acc + (size_t)j * kAccStride, kOne + (unsigned long long)v);
        }
        if (tid == kNC - 1) {
          const long long v = scale_x2 != 0.0 ? __double2ll_rn((double)misc->x2_part * scale_x2) : 0ll;
          red_add_u64(acc + (size_t)k * kAccStride, kOne + (unsigned long long)v);
        }
      }
    }
    if (contrib_p && tid == kNC - 2) {
      float sr = 0.f;   // fixed order: the sum does not depend on which warp finished first
#pragma unroll
      for (int w = 0; w < kNW; ++w) sr += misc->sr[w];
      // at most 2^45 per CTA, so the sum of all CTAs stays below 2^53; a partial that large
      // (||r||^2 > 2 ||x||^2) fires for every sensible eps
      double vd = (double)sr * pow2d(44 - e_p);
      if (!(vd < 35184372088832.0)) vd = 35184372088832.0;
      if (!(vd >= 0.0)) vd = 0.0;
      red_add_u64(r2word_p, kOne + (unsigned long long)__double2ll_rn(vd));
    }
    tr.mark(4);

    // ---- E. wait until every contributing CTA has been added.  One thread watches one word
    //      (thousands of pollers on the accumulators would delay the very atomics they wait
    //      for); then every thread validates its own word, which is normally complete by then.
    if (gsi) {
      if (tid == 0) (void)poll_acc(acc + (size_t)(k - 1) * kAccStride, (unsigned)n_contrib, p, misc);
      csync();
      if (*abort) return;
#pragma unroll 1
      for (int j = tid; j < k; j += kNC) {
        const long long val = poll_acc(acc + (size_t)j * kAccStride, (unsigned)n_contrib, p, misc);
        s_c[j] = (float)((double)val * inv_scale);
      }
      if (tid == kNC - 1) {
        const long long val = poll_acc(acc + (size_t)k * kAccStride, (unsigned)n_contrib, p, misc);
        const double amax = (double)__uint_as_float(misc->amax_bits);
        const double x2 = nonfinite ? __longlong_as_double(0x7ff8000000000000ll)
                          : val > 0 ? (double)val * pow2d(exp_above(amax * amax * (double)g.p_rows) - 43)
                                    : 0.0;
        misc->x2 = x2;
        // every CTA decides this group's gate in the next tick from the published value
        if (lc == 0)
          st_relaxed_u64(g.pub, ((unsigned long long)__double_as_longlong(x2) & ~(1ull << 63)) |
                                    ((unsigned long long)tag << 63));
      }
    }
    // the previous phase's gates: one thread per group collects ||r||^2 and ||x||^2 and decides
    if (len_p > 0 && (tid == kNC - 3 || tid == kNC - 4) && kNC - 3 - tid < len_p) {
      const int u = kNC - 3 - tid;
      const PersistGroup* gp = p.groups + g_p + u;
      const unsigned fl = __ldg(&gp->flags);
      if (!(fl & GSI_FLAG_DENSE)) {
        const int k_u = __ldg(&gp->k), d_u = __ldg(&gp->d), pr_u = __ldg(&gp->p_rows);
        const unsigned n_u = (unsigned)((d_u + pr_u - 1) / pr_u);
        const unsigned long long* acc_u =
            reinterpret_cast<const unsigned long long*>(__ldg(reinterpret_cast<const unsigned long long*>(&gp->acc))) +
            (size_t)parity * (k_u + 2) * kAccStride;
        const unsigned long long* pub_u =
            reinterpret_cast<const unsigned long long*>(__ldg(reinterpret_cast<const unsigned long long*>(&gp->pub)));
        const long long val = poll_acc(acc_u + (size_t)(k_u + 1) * kAccStride, n_u, p, misc);
        unsigned long long w = 0;
        unsigned it = 0;
        for (;;) {
          w = ld_relaxed_u64(pub_u);
          if ((unsigned)(w >> 63) == tag) break;
          if (++it > p.spin_limit || ((it & 1023u) == 0 && *abort)) {
            if (!*abort) fail(p, misc);
            break;
          }
        }
        const double x2 = __longlong_as_double((long long)(w & ~(1ull << 63)));
        const bool finite = x2 == x2;
        const double r2 = (double)val * pow2d((x2 > 0.0 ? exp_above(x2) : 0) - 44);
        const double eps = (double)__ldg(&gp->eps);
        // ||r|| < eps ||x||  <=>  ||r||^2 < eps^2 ||x||^2  (both sides >= 0); false for x = 0
        const bool fast = finite && (r2 < eps * eps * x2);
        misc->fire[(t & 1) * 2 + u] = (!fast && finite && !(fl & GSI_FLAG_STATIC_PROJECTION)) ? 1 : 0;
        if (cta == 0) {
          const size_t at = ((size_t)slot_io * p.log_step_stride + (g_p + u)) * p.n_tokens + p.token;
          p.gate_log[at] = fast ? 0 : 1;
          if (p.rho_log)
            p.rho_log[at] = finite ? (float)sqrt(r2 / x2) : __int_as_float(0x7fc00000);
        }
      }
    }
    csync();
    tr.mark(5);
    if (*abort) return;

    // ---- F. hand the decision to the producer; a gated group's r and image rows must be
    //      visible grid-wide before its W rows are streamed in the next tick: release fence
    //      and arrival now, the wait comes then
    const unsigned mask_p = (unsigned)misc->fire[(t & 1) * 2] | ((unsigned)misc->fire[(t & 1) * 2 + 1] << 1);
    if (tid == 0 && t >= 1) {
      misc->decision[(t - 1) & 3] = ((unsigned)t << 8) | mask_p;
#pragma unroll 1
      for (int u = 0; u < len_p; ++u)
        if (mask_p & (1u << u)) {
          __threadfence();
          red_relaxed_u32(p.groups[g_p + u].bar + 2 + parity, 1u);
        }
    }
    const double x2_own = gsi ? misc->x2 : 0.0;

    // ---- G. pass 2: residual rows of the basis chunks (still in the ring)
    const int itemsP = (prow + 7) >> 3, itemsO = (orow + 7) >> 3;
    const int padP = ((itemsP + (1 << rpp_log2) - 1) >> rpp_log2) << rpp_log2;
    const int padO = ((itemsO + (1 << rpp_log2) - 1) >> rpp_log2) << rpp_log2;
    if (gsi) {
      float sr = row_items<false>(q, rg, n_p0, pchunks, prow, 0, padP, s_c, s_x, g.r + s.p0, false, ok);
      sr = warp_sum(sr);
      if (lane == 0) misc->sr[warp] = sr;
      rg.n += pchunks;
      tr.mark(6);
    }

    // ---- H. gated residuals of the phase before the previous one
    if (mask_pp) {
#pragma unroll 1
      for (int u = 0; u < len_pp && ok; ++u) {
        if (!(mask_pp & (1u << u))) continue;
        const PersistGroup& gg = p.groups[g_pp + u];
        if (tid == 0) {
          grid_wait(gg.bar + 2 + parity, (unsigned)G, p, misc);
          __threadfence();
        }
        csync();
        if (*abort) return;
        ok = w_stream(p, gg, gg.r, gg.y + (size_t)p.token * gg.O, false, smem, ctx, misc);
      }
      tr.mark(7);
    }

    // ---- I. image rows; or, for a dense group, its whole W stream and a grid barrier that
    //      keeps the groups of a dense stack in model order
    if (gsi) {
      const unsigned n_o0 = rg.n;
      ok = ok && chunks_landed(rg, n_o0, ochunks, abort);
      tr.mark(8);
      (void)row_items<true>(q, rg, n_o0, ochunks, orow, padP, padO, s_c, s_x,
                            g.y + (size_t)p.token * g.O + s.o0, nonfinite, ok);
      rg.n += ochunks;
      if (!ok && !*abort) fail(p, misc);
      tr.mark(9);
    } else if (dense) {
      const float* x = g.x + (long long)slot_io * g.x_step_stride + (size_t)p.token * g.d;
      ok = ok && w_stream(p, g, x, g.y + (size_t)p.token * g.O, true, smem, ctx, misc);
      if (tid == 0) {
        red_relaxed_u32(g.bar + parity, 1u);
        grid_wait(g.bar + parity, (unsigned)G, p, misc);
        if (cta == 0)
          p.gate_log[((size_t)slot_io * p.log_step_stride + gi) * p.n_tokens + p.token] = 1;
      }
      csync();
      tr.mark(10);
    }
    if (*abort) return;

    contrib_p = gsi && prow > 0;
    if (gsi) {
      e_p = x2_own > 0.0 ? exp_above(x2_own) : 0;
      r2word_p = acc + (size_t)(k + 1) * kAccStride;
    }
    g_pp = g_p;
    len_pp = len_p;
    mask_pp = mask_p;
    g_p = gi;
    len_p = len;
    gi += len;
  }
  // Every CTA read the counters at its start and has since taken part in the
  // last group's exchange, so they may advance now.
  if (cta == 0 && tid == 0 && ok && !*abort) {
    *p.epoch = epoch + 1;
    if (p.use_counter && p.advance) *p.step = step + 1;
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
