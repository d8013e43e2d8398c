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
constexpr int kNB = 32;                     // chunks in flight at most (one barrier pair each)
constexpr int kChunk = 16384;               // largest chunk
constexpr int kSlice = 4096;                // columns of W per staged slice of r
constexpr int kBoxCols = kPersistBoxCols;
constexpr unsigned kLocalSpinLimit = 1u << 20;   // waits inside the CTA (ring, producer hand-off)
constexpr int kCountShift = 54;
constexpr unsigned long long kOne = 1ull << kCountShift;

// What one CTA does in one tick of a launch, worked out once at the start of the launch.
struct Plan {
  short gi;        // the group whose fast path (or dense stream) this CTA runs in this tick
  short gi0;       // first group of the tick's phase
  unsigned char len, next_len;   // groups in this phase and in the next
  unsigned char kind;            // 0 nothing (closing ticks), 1 gated subspace group, 2 dense group
  unsigned char zeroer;          // this CTA clears the group's counters for the next launch
  short prow, orow;              // rows of the basis slab and of the image slab
  short pchunks, ochunks;        // ... and their ring chunks
  int p0, o0;                    // first rows
  short lc, n_contrib;           // index within the group's share of the grid; CTAs that own basis rows
  int pad;
};
static_assert(sizeof(Plan) == 32, "one plan record");

// shared memory map (bytes)
constexpr int kOffBar = 0;          // full[kNB], empty[kNB]
constexpr int kOffLin = 512;        // producer: ring position (bytes placed before it) of every chunk in flight (kNB words)
constexpr int kOffOff = 640;        // offset of every chunk in flight within the ring (kNB words), for the consumers
constexpr int kOffMisc = 768;       // scalars
constexpr int kOffTrace = 1024;     // cycle counters of the trace (16 words)
constexpr int kOffX = 1280;         // x of this CTA's basis rows, two buffers (kPersistMaxPRows floats each)
constexpr int kOffC = kOffX + 2 * kPersistMaxPRows * 4;   // c (512 floats)
constexpr int kOffFx = kOffC + 2048;                      // fixed-point partial c and ||x||^2, source of the bulk reduction (514 words)
constexpr int kOffPlan = kOffFx + 4224;                   // the launch's plan (kPersistMaxTicks records)
constexpr int kOffDesc = kOffPlan + kPersistMaxTicks * 32;   // 8 group descriptors, 256 B each
constexpr int kDescSlots = 8;
constexpr int kOffRed = kOffDesc + kDescSlots * 256;      // cross-warp scratch of pass 1 ((kNW-1)*512 floats) ...
constexpr int kOffRs = kOffRed;                           // ... which the W stream reuses for its slice of r (16 KB)
constexpr int kOffYacc = kOffRed + (kNW - 1) * 512 * 4;   // per-row accumulators (kPersistMaxORows floats)
constexpr int kOffRing = ((kOffYacc + kPersistMaxORows * 4 + 1023) / 1024) * 1024;
constexpr int kRingBytes = (232448 - kOffRing) / 1024 * 1024;
constexpr int kSmemBytes = kOffRing + kRingBytes;
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 CTA");
static_assert(kOffFx % 16 == 0 && kOffPlan % 16 == 0 && kOffDesc % 16 == 0, "alignment");
static_assert(kSlice * 4 <= (kNW - 1) * 512 * 4, "the staged slice fits the scratch it shares");
static_assert(sizeof(PersistGroup) <= 256 && sizeof(PersistGroup) % 4 == 0, "descriptor slot");
static_assert(kPersistBoxRowsMax * kBoxCols * 2 <= kChunk, "a box fits a chunk");
static_assert(kPersistBoxRowsMax == 2 * kNW, "two rows of a box per consumer warp");
constexpr int kDescWords = (int)(sizeof(PersistGroup) / 4);

struct Misc {
  int abort;
  unsigned amax_bits;       // max |x| of this phase's group (>= 0x7f800000: a non-finite token)
  float x2_part[2];         // this CTA's sum of x^2 over its rows, by tick parity
  int fire[4];              // decisions on the previous phase's groups, by tick parity: 1 = stream W
  double x2;                // ||x||^2 of this phase's group
  float sr[kNW];            // per-warp partial ||r||^2 of this phase
  volatile unsigned decision[4];   // hand-off to the producer: (phase + 1) << 8 | fire mask
};
static_assert(sizeof(Misc) <= kOffTrace - kOffMisc, "scalars");

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
// Element-wise atomic add of `bytes` / 8 64-bit words from shared to global memory by the bulk
// copy engine (each element's addition is a relaxed atomic at the L2).
__device__ __forceinline__ void bulk_reduce_add_u64(void* gdst, const void* ssrc, uint32_t bytes) {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.u64 [%0], [%1], %2;" ::"l"(gdst),
               "r"(smem_u32(ssrc)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_reduce_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
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

// Records the time-out; `site` (which wait gave up, for diagnosis) goes to the word after
// the status word, first failure only.
__device__ __forceinline__ void fail(const PersistParams& p, Misc* misc, int site) {
  misc->abort = 1;
  atomicExch(p.status, (int)GSI_ERR_TIMEOUT);
  atomicCAS(p.status + 1, 0, site);
}

// Optional cycle trace (thread 0 of every CTA; sections of the per-phase pipeline, summed
// over phases in shared memory and added to p.trace when the CTA ends); p.trace == nullptr
// disables it.
struct Trace {
  unsigned long long* acc;   // shared
  long long t;
  __device__ __forceinline__ void start(const PersistParams& p, unsigned char* smem) {
    acc = (threadIdx.x == 0 && p.trace) ? reinterpret_cast<unsigned long long*>(smem + kOffTrace) : nullptr;
    if (acc) {
      for (int i = 0; i < 16; ++i) acc[i] = 0ull;
      t = clock64();
    }
  }
  __device__ __forceinline__ void mark(int section) {
    if (acc) {
      const long long now = clock64();
      acc[section] += (unsigned long long)(now - t);
      t = now;
    }
  }
  __device__ __forceinline__ void flush(const PersistParams& p) {
    if (acc)
      for (int i = 0; i < 16; ++i) p.trace[(size_t)blockIdx.x * 16 + i] += acc[i];
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

// ------------------------------------------------------------------ the ring
// Chunks of any size up to 16 KB are packed back to back in a circular byte buffer (a chunk
// never wraps: the tail of the buffer is skipped instead).  `lin` counts bytes placed so far,
// skipped tails included, so lin % kRingBytes is the physical offset; chunk n uses barrier
// pair n % kNB.  The producer publishes the offset of chunk n in s_off[n % kNB] before it arms
// the chunk's "full" barrier; producer and consumers walk the same sequence of chunks, so a
// consumer needs only the sequence number.
struct Producer {
  uint64_t* full;
  uint64_t* empty;
  unsigned char* base;
  unsigned* s_lin;     // shared: start (lin) of every chunk in flight
  unsigned* s_off;     // shared: its offset in the ring
  unsigned n;          // sequence number of the next chunk
  unsigned lin;        // bytes placed so far
  unsigned tail_n;     // oldest chunk not yet given back by the consumers
  unsigned tail_lin;   // where it starts
};

// Reserve `bytes` for chunk n: waits (bounded) until the consumers have given back every
// older chunk that still overlaps the place, and a barrier pair is free.  Returns the
// offset, or 0xffffffff when a wait gave up.
__device__ __forceinline__ unsigned producer_acquire(Producer& pr, unsigned bytes, volatile int* abort) {
  unsigned off = pr.lin % (unsigned)kRingBytes;
  if (off + bytes > (unsigned)kRingBytes) {
    pr.lin += (unsigned)kRingBytes - off;
    off = 0;
  }
  const unsigned start = pr.lin;
  pr.lin += bytes;
  while (pr.n - pr.tail_n >= (unsigned)kNB ||
         (pr.tail_n < pr.n && pr.lin - pr.tail_lin > (unsigned)kRingBytes)) {
    if (!mbar_wait(&pr.empty[pr.tail_n % kNB], (pr.tail_n / kNB) & 1u, abort)) return 0xffffffffu;
    ++pr.tail_n;
    pr.tail_lin = pr.tail_n < pr.n ? pr.s_lin[pr.tail_n % kNB] : start;
  }
  if (pr.tail_n == pr.n) pr.tail_lin = start;
  pr.s_lin[pr.n % kNB] = start;
  pr.s_off[pr.n % kNB] = off;
  return off;
}

// The W boxes of one group for this CTA, in the order the consumers take them: column
// slices of 4096 outermost (one staged slice of r serves them), then maps, then row blocks,
// then the 256-column boxes of the slice.
__device__ __forceinline__ bool produce_w(const PersistGroup& g, Producer& pr, volatile int* abort) {
  const int cta = blockIdx.x;
  const int nsl = (g.d + kSlice - 1) / kSlice;
  for (int sl = 0; sl < nsl; ++sl) {
    const int c0 = sl * kSlice, ncb = (min(kSlice, g.d - c0) + kBoxCols - 1) / kBoxCols;
    for (int j = 0; j < g.n_maps; ++j) {
      const int dout = g.off[j + 1] - g.off[j], rows = g.w_rows[j], rb = g.w_rb[j];
      const int row0 = cta * rows;
      const int live = min(rows, dout - row0);
      const char* tm = static_cast<const char*>(g.tmW) + (size_t)j * kPersistTmapBytes;
      const uint32_t bytes = (uint32_t)rb * kBoxCols * 2;
      for (int b = 0; b * rb < live; ++b) {
        for (int cb = 0; cb < ncb; ++cb) {
          const unsigned off = producer_acquire(pr, bytes, abort);
          if (off == 0xffffffffu) return false;
          uint64_t* fb = &pr.full[pr.n % kNB];
          mbar_expect_tx(fb, bytes);
          tma_box_g2s(pr.base + off, tm, c0 + cb * kBoxCols, row0 + b * rb, fb);
          ++pr.n;
        }
      }
    }
  }
  return true;
}

// Rows [a, b) of a row-major [rows][k] bf16 matrix as chunks of whole rows.
__device__ __forceinline__ bool produce_rows(const uint16_t* base, int k, int a, int b, Producer& pr,
                                             volatile int* abort) {
  const int rc = kChunk / (k * 2);
  for (int r = a; r < b; r += rc) {
    const int rows = min(rc, b - r);
    const uint32_t bytes = (uint32_t)rows * k * 2;
    const unsigned off = producer_acquire(pr, bytes, abort);
    if (off == 0xffffffffu) return false;
    uint64_t* fb = &pr.full[pr.n % kNB];
    mbar_expect_tx(fb, bytes);
    bulk_g2s(pr.base + off, base + (size_t)r * k, bytes, fb);
    ++pr.n;
  }
  return true;
}

__device__ void producer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  Producer pr;
  pr.full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  pr.empty = pr.full + kNB;
  pr.base = smem + kOffRing;
  pr.s_lin = reinterpret_cast<unsigned*>(smem + kOffLin);
  pr.s_off = reinterpret_cast<unsigned*>(smem + kOffOff);
  pr.n = 0;
  pr.lin = 0;
  pr.tail_n = 0;
  pr.tail_lin = 0;
  volatile int* abort = &misc->abort;
  const int cta = blockIdx.x;
  bool ok = true;
  // ticks: tick t runs phase t (while there is one) and the gated residuals of phase t - 2;
  // the work of a tick, in ring order: basis slab, W boxes of the gated groups, image slab
  // (or the W boxes of a dense group)
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
      ok = produce_rows(g->P, g->k, s.p0, s.p1, pr, abort);
    }
    unsigned wmask = 0;
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
      wmask = v & 3u;
    }
    // one call site for every W stream of the tick: the gated groups, then a dense group
#pragma unroll 1
    for (int u = 0; ok && u < 3; ++u) {
      const PersistGroup* gw = nullptr;
      if (u < 2) {
        if (u < len_pp && (wmask & (1u << u))) gw = &p.groups[g_pp + u];
      } else if (dense) {
        gw = g;
      }
      if (gw) ok = produce_w(*gw, pr, abort);
    }
    if (ok && own && !dense) ok = produce_rows(g->WP, g->k, s.o0, s.o1, pr, abort);
    g_pp = g_p;
    len_pp = len_p;
    g_p = gi;
    len_p = len;
    gi += len;
  }
  if (!ok && !*abort) fail(p, misc, 1);
  // Every copy issued must have landed before the CTA may give up its shared
  // memory: wait (bounded) for the last kNB chunks.
  {
    const unsigned first = pr.n > (unsigned)kNB ? pr.n - kNB : 0;
    for (unsigned c = first; c < pr.n; ++c) {
      const unsigned slot = c % kNB, ph = (c / kNB) & 1u;
      for (unsigned it = 0; it < kLocalSpinLimit; ++it)
        if (mbar_try(&pr.full[slot], ph)) break;
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
      if (!*abort) fail(p, misc, 2);
      return false;
    }
  }
  return true;
}

// Chunks [n0, n0 + count) have landed (lane c waits for chunk c, all waits in flight together).
__device__ __forceinline__ bool chunks_landed(unsigned char* smem, unsigned n0, int count,
                                              volatile int* abort) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  const int lane = threadIdx.x & 31;
  bool mine_ok = true;
  if (lane < count) {
    const unsigned seq = n0 + lane;
    mine_ok = mbar_wait(&full[seq % kNB], (seq / kNB) & 1u, abort);
  }
  return __all_sync(0xffffffffu, mine_ok);
}

// ---- W stream: y_rows (+)= W_rows . src (src = r of a gated group, or x for the dense
// baseline), boxes taken from the ring in the producer's order.  `n` is the consumers' chunk
// sequence number.  Returns false when a wait gave up.
__device__ __forceinline__ bool w_stream(const PersistParams& p, const PersistGroup& g, const float* src,
                                         float* y, bool dense, unsigned char* smem, unsigned& n,
                                         Misc* misc) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kNB;
  const unsigned* s_off = reinterpret_cast<const unsigned*>(smem + kOffOff);
  unsigned char* ring = smem + kOffRing;
  float* s_rs = reinterpret_cast<float*>(smem + kOffRs);
  float* s_yacc = reinterpret_cast<float*>(smem + kOffYacc);
  volatile int* abort = &misc->abort;
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
          const unsigned slot = n % kNB, ph = (n / kNB) & 1u;
          ++n;
          if (ok && !mbar_wait(&full[slot], ph, abort)) ok = false;
          if (ok && mine) {
            const uint4* tile = reinterpret_cast<const uint4*>(ring + s_off[slot]);
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
          if (ok && lane == 0) mbar_arrive(&empty[slot]);
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
  if (!ok && !*abort) fail(p, misc, 3);
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

// kPairs = false compiles the pair logic out: stacks without concurrent groups run a smaller
// loop (the per-phase code has to stay short: it is executed once per phase, straight through,
// so its length is paid in instruction fetches).  kK != 0 is a build for stacks whose groups all
// have rank kK (shifts, strides and loop bounds become constants); kK = 0 reads the rank from
// the descriptor.
template <bool kPairs, int kK>
__device__ void consumer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  uint64_t* empty = reinterpret_cast<uint64_t*>(smem + kOffBar) + kNB;
  const unsigned* s_off = reinterpret_cast<const unsigned*>(smem + kOffOff);
  unsigned char* ring = smem + kOffRing;
  float* s_xb = reinterpret_cast<float*>(smem + kOffX);
  float* s_c = reinterpret_cast<float*>(smem + kOffC);
  unsigned long long* s_fx = reinterpret_cast<unsigned long long*>(smem + kOffFx);
  float* s_red = reinterpret_cast<float*>(smem + kOffRed);
  Plan* plan = reinterpret_cast<Plan*>(smem + kOffPlan);
  volatile int* abort = &misc->abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  constexpr int kStatWarp = kNW - 1;   // statistics of x and the collection of max|x|; the others run pass 1
  constexpr int kP1 = kNW - 1;         // warps of pass 1

  unsigned n = 0;   // chunk sequence number: advances exactly as in producer()
  const int step = p.use_counter ? *p.step : 0;
  const int slot_io = step % p.n_steps;
  const int epoch = *p.epoch;
  const unsigned parity = (unsigned)epoch & 1u, tag = ((unsigned)epoch + 1u) & 1u;
  const int n_ticks = p.n_phases + 2;
  Trace tr;
  tr.start(p, smem);

  auto desc = [&](int i) -> const PersistGroup& {
    return *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (i & (kDescSlots - 1)) * 256);
  };
  // groups [g0, g0 + cnt) from the device table into their slots (threads 0 .. cnt*kDescWords-1)
  auto desc_load = [&](int g0, int cnt) -> uint32_t {
    return tid < cnt * kDescWords ? __ldg(reinterpret_cast<const uint32_t*>(p.groups + g0) + tid) : 0u;
  };
  auto desc_store = [&](int g0, int cnt, uint32_t w) {
    if (tid < cnt * kDescWords) {
      const int j = tid >= kDescWords ? 1 : 0;
      reinterpret_cast<uint32_t*>(smem + kOffDesc + ((g0 + j) & (kDescSlots - 1)) * 256)[tid - j * kDescWords] = w;
    }
  };
  // one warp: request this CTA's rows of x for tick `tt` into buffer tt & 1
  auto request_x = [&](int tt) {
    const Plan& pn = plan[tt];
    if (pn.kind != 1) return;
    const PersistGroup& gn = desc(pn.gi);
    const float* src = gn.x + (long long)slot_io * gn.x_step_stride + (size_t)p.token * gn.d + pn.p0;
    float* dst = s_xb + (tt & 1) * kPersistMaxPRows;
    for (int i = lane; i < pn.prow; i += 32) cp_async4(dst + i, src + i);
  };

  // the statistics warp: max |x| and sum x^2 over this CTA's rows of x for tick `tt` (the rows
  // have been requested); the maximum is published at once as a tagged word, the sum is kept
  // for the tick's exchange
  auto publish_stats = [&](int tt) {
    const Plan& pn = plan[tt];
    if (pn.kind != 1) return;
    cp_async_wait_all();
    __syncwarp();
    const float* sx = s_xb + (tt & 1) * kPersistMaxPRows;
    float amax = 0.f, s2 = 0.f;
#pragma unroll 1
    for (int i = lane; i < pn.prow; i += 32) {
      const float v = sx[i];
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
      if (pn.prow > 0) st_relaxed_u32(desc(pn.gi).xmax + pn.lc, bits | (tag << 31));
      misc->x2_part[tt & 1] = s2;
    }
  };

  // ---- the plan of this launch for this CTA, one thread per tick
#pragma unroll 1
  for (int t = tid; t < n_ticks; t += kNC) {
    Plan pl{};
    pl.gi = pl.gi0 = -1;
    if (t < p.n_phases) {
      const int gi0 = __ldg(p.phase_first + t);
      const PersistGroup* ga = p.groups + gi0;
      const int len = kPairs ? __ldg(&ga->phase_len) : 1;
      int gi = gi0;
      if (kPairs && len == 2 && cta >= __ldg(&ga->cta0) + __ldg(&ga->ncta)) gi = gi0 + 1;
      const PersistGroup* g = p.groups + gi;
      const bool dense = __ldg(&g->flags) & GSI_FLAG_DENSE;
      pl.gi = (short)gi;
      pl.gi0 = (short)gi0;
      pl.len = (unsigned char)len;
      pl.next_len = (unsigned char)(kPairs ? __ldg(&ga->next_len) : min(__ldg(&ga->next_len), 1));
      pl.kind = dense ? 2 : 1;
      const int lc = cta - __ldg(&g->cta0), ncta = __ldg(&g->ncta);
      pl.lc = (short)lc;
      pl.zeroer = lc == gi % ncta;
      if (!dense) {
        const int d = __ldg(&g->d), O = __ldg(&g->O), pr = __ldg(&g->p_rows), orw = __ldg(&g->o_rows);
        const int k = kK ? kK : __ldg(&g->k);
        const int rc = kChunk / (k * 2);
        const int p0 = min(d, lc * pr), p1 = min(d, p0 + pr);
        const int o0 = min(O, lc * orw), o1 = min(O, o0 + orw);
        pl.p0 = p0;
        pl.o0 = o0;
        pl.prow = (short)(p1 - p0);
        pl.orow = (short)(o1 - o0);
        pl.pchunks = (short)((p1 - p0 + rc - 1) / rc);
        pl.ochunks = (short)((o1 - o0 + rc - 1) / rc);
        pl.n_contrib = (short)__ldg(&g->n_contrib);
      }
    }
    plan[t] = pl;
  }
  // the first phase's descriptors (the second slot is used only if the phase is a pair)
  desc_store(0, min(p.n_groups, 2), desc_load(0, min(p.n_groups, 2)));
  csync();
  if (warp == kStatWarp) {
    request_x(0);
    cp_async_commit();
    publish_stats(0);
  }

  unsigned mask_pp = 0;          // gates that fired in the phase before the previous one
  bool contrib_p = false;        // this CTA holds a partial ||r||^2 of the previous phase
  int e_p = 0;                   // ... scaled by 2^(44 - e_p)
  unsigned long long* r2word_p = nullptr;
  bool ok = true;

#pragma unroll 1
  for (int t = 0; t < n_ticks && ok; ++t) {
    const Plan pl = plan[t];
    const bool gsi = pl.kind == 1, dense = pl.kind == 2;
    const PersistGroup& g = desc(pl.gi);        // read only when the tick has a group
    const int k = gsi ? (kK ? kK : g.k) : 0;
    const int prow = pl.prow, orow = pl.orow, pchunks = pl.pchunks, ochunks = pl.ochunks;
    const int n_contrib = pl.n_contrib, lc = pl.lc;
    const int len_p = t >= 1 ? plan[t - 1].len : 0, g_p = t >= 1 ? plan[t - 1].gi0 : 0;
    float* s_x = s_xb + (t & 1) * kPersistMaxPRows;
    unsigned long long* acc = gsi ? g.acc + (size_t)parity * (k + 4) : nullptr;
    const int tp = (t & 1) * 2;

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

    // the next phase's descriptors: requested now, stored after pass 1
    const uint32_t desc_word = desc_load(pl.gi0 + pl.len, pl.next_len);

    // ---- A. this CTA's rows of x have arrived (requested one phase ago); the bulk reduction
    //      of the previous tick has read its source
    if (tid == 0) {
      bulk_reduce_wait_read();
      misc->fire[tp] = misc->fire[tp + 1] = 0;
    }
    if (pl.zeroer) {  // this CTA clears the group's counters for the next launch
      if (gsi) {
#pragma unroll 1
        for (int j = tid; j < k + 4; j += kNC) g.acc[(size_t)(parity ^ 1u) * (k + 4) + j] = 0ull;
      }
      if (tid < 2) g.bar[2 * tid + (parity ^ 1u)] = 0u;
    }
    csync();
    tr.mark(0);

    const unsigned n_p0 = n;
    n += pchunks;
    if (gsi) {
      if (warp == kStatWarp) {
        // ---- the group's max |x|: collect the tagged words of all contributing CTAs (lane l
        //      owns words l, l+32, ...; they were published during the previous tick) while
        //      the other warps run pass 1
        unsigned m = 0, it = 0;
        bool done = false;
        while (!done) {
          bool all = true;
          m = 0;
#pragma unroll
          for (int i = 0; i < kPersistMaxGrid / 32; ++i) {   // all loads in flight together
            const int w_i = lane + 32 * i;
            if (w_i < n_contrib) {
              const unsigned w = ld_relaxed_u32(g.xmax + w_i);
              all = all && ((w >> 31) == tag);
              m = max(m, w & 0x7fffffffu);
            }
          }
          done = __all_sync(0xffffffffu, all);
          if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
            if (!*abort && lane == 0) fail(p, misc, 4);
            break;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) misc->amax_bits = m;
      } else {
        // ---- B. pass 1: partial c over this CTA's basis rows
        ok = chunks_landed(smem, n_p0, pchunks, abort);
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
            const uint4* tile = reinterpret_cast<const uint4*>(ring + s_off[(n_p0 + ci) % kNB]);
            const int r_lo = ci << q.rc_log2, rows = min(rc, prow - r_lo);
#pragma unroll 2
            for (int row = (warp << rpp_log2) + q.sub; row < rows; row += kP1 << rpp_log2) {
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
        if (!ok && !*abort) fail(p, misc, 5);
      }
    }
    desc_store(pl.gi0 + pl.len, pl.next_len, desc_word);
    csync();
    tr.mark(2);
    if (*abort) return;
    // the next phase's rows of x travel while this phase runs its exchange (its descriptors
    // are in place now) ...
    if (warp == kStatWarp && t + 1 < n_ticks) {
      request_x(t + 1);
      cp_async_commit();
    }

    // ---- D. the exchange: this phase's partial c and ||x||^2 as ONE bulk reduction of k + 2
    //      fixed-point words into the group's accumulators, the previous phase's ||r||^2 as
    //      one atomic
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
          for (int w = 0; w < kP1; ++w) sum += s_red[w * 512 + j];
          const long long v = scale != 0.0 ? __double2ll_rn((double)sum * scale) : 0ll;
          s_fx[j] = kOne + (unsigned long long)v;
        }
        if (tid == kNC - 1) {
          const long long v = scale_x2 != 0.0 ? __double2ll_rn((double)misc->x2_part[t & 1] * scale_x2) : 0ll;
          s_fx[k] = kOne + (unsigned long long)v;
          s_fx[k + 1] = 0ull;
        }
      }
    }
    csync();
    if (tid == 0 && gsi && prow > 0) bulk_reduce_add_u64(acc, s_fx, (uint32_t)(k + 2) * 8);
    if (contrib_p && tid == 32) {
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
    tr.mark(3);

    // ---- E. wait until every contributing CTA has been added: warp 0 polls the accumulators
    //      of c (contiguous: lane l owns words l, l+32, ..., all its loads in flight together,
    //      one round trip per attempt), warp 1 the scalars: lane 0 this phase's ||x||^2, lanes
    //      1+2u / 2+2u the previous phase's ||r||^2 and published ||x||^2 of its group u.
    if (gsi && warp == 0) {
      unsigned it = 0;
      bool done = false;
      while (!done) {
        bool all = true;
#pragma unroll 8
        for (int j = lane; j < k; j += 32) {
          const unsigned long long w = ld_relaxed_u64(acc + j);
          all = all && ((unsigned)((w + (kOne >> 1)) >> kCountShift) == (unsigned)n_contrib);
          const long long val = (long long)(w - ((unsigned long long)n_contrib << kCountShift));
          s_c[j] = (float)((double)val * inv_scale);
        }
        done = __all_sync(0xffffffffu, all);
        if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
          if (!*abort && lane == 0) fail(p, misc, 6);
          break;
        }
      }
    }
    if (warp == 1) {
      // what this lane watches: an accumulator (count in the upper bits) or a tagged word
      const int u = (lane - 1) >> 1;
      const bool settle = lane >= 1 && lane <= 4 && u < len_p && !(desc(g_p + u).flags & GSI_FLAG_DENSE);
      const PersistGroup& gs = desc(g_p + (u & 1));   // read only when `settle`
      const bool w_x2 = gsi && lane == 0;
      const bool w_r2 = settle && (lane & 1), w_pub = settle && !(lane & 1);
      const unsigned long long* wp = w_x2   ? acc + k
                                     : w_r2 ? gs.acc + (size_t)parity * (gs.k + 4) + gs.k + 2
                                            : gs.pub;
      const unsigned want = w_x2 ? (unsigned)n_contrib : (unsigned)gs.n_contrib;
      unsigned long long w = 0;
      unsigned it = 0;
      bool done = false;
      while (!done) {
        bool mine = true;
        if (w_x2 || w_r2) {
          w = ld_relaxed_u64(wp);
          mine = (unsigned)((w + (kOne >> 1)) >> kCountShift) == want;
        } else if (w_pub) {
          w = ld_relaxed_u64(wp);
          mine = (unsigned)(w >> 63) == tag;
        }
        done = __all_sync(0xffffffffu, mine);
        if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
          if (!*abort && lane == 0) fail(p, misc, 7);
          break;
        }
      }
      if (w_x2) {
        const long long val = (long long)(w - ((unsigned long long)n_contrib << kCountShift));
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
      // the previous phase's gates: the lane that holds ||r||^2 of group u takes ||x||^2 from
      // its neighbour and decides
      const unsigned long long w_nb = __shfl_down_sync(0xffffffffu, w, 1);
      if (w_r2) {
        const long long val = (long long)(w - ((unsigned long long)want << kCountShift));
        const double x2 = __longlong_as_double((long long)(w_nb & ~(1ull << 63)));
        const bool finite = x2 == x2;
        const int ex = x2 > 0.0 ? exp_above(x2) : 0;
        const double r2 = (double)val * pow2d(ex - 44);
        const double eps = (double)gs.eps;
        // ||r|| < eps ||x||  <=>  ||r||^2 < eps^2 ||x||^2  (both sides >= 0); false for x = 0
        const bool fast = finite && (r2 < eps * eps * x2);
        misc->fire[tp + u] = (!fast && finite && !(gs.flags & GSI_FLAG_STATIC_PROJECTION)) ? 1 : 0;
        if (cta == 0) {
          const size_t at = ((size_t)slot_io * p.log_step_stride + (g_p + u)) * p.n_tokens + p.token;
          p.gate_log[at] = fast ? 0 : 1;
          if (p.rho_log)   // both operands scaled into the float range: ||r||^2 2^-e and ||x||^2 2^-e
            p.rho_log[at] = finite ? sqrtf(__fdividef((float)((double)val * 5.6843418860808015e-14),
                                                      (float)(x2 * pow2d(-ex))))
                                   : __int_as_float(0x7fc00000);
        }
      }
    }
    csync();
    tr.mark(4);
    if (*abort) return;

    // ---- F. hand the decision to the producer; a gated group's r and image rows must be
    //      visible grid-wide before its W rows are streamed in the next tick: release fence
    //      and arrival now, the wait comes then
    const unsigned mask_p = (unsigned)misc->fire[tp] | ((unsigned)misc->fire[tp + 1] << 1);
    if (tid == 0 && t >= 1) {
      misc->decision[(t - 1) & 3] = ((unsigned)t << 8) | mask_p;
#pragma unroll 1
      for (int u = 0; u < len_p; ++u)
        if (mask_p & (1u << u)) {
          __threadfence();
          red_relaxed_u32(desc(g_p + u).bar + 2 + parity, 1u);
        }
    }
    const double x2_own = gsi ? misc->x2 : 0.0;
    // ... and their statistics are published a row pass ahead of the next phase's exchange
    if (warp == kStatWarp && t + 1 < n_ticks) publish_stats(t + 1);

    // ---- G / I. the row passes, one copy of the code for both: part 0 the residual rows of
    //      the basis slab (still in the ring), part 1 the image rows.  Items of eight rows
    //      (one lane group each) are dealt round-robin over the joint numbering of both
    //      parts, so the warps are loaded evenly.  Every warp gives every chunk back once.
    // ---- H (between them). the W streams of the tick, one call site: the gated residuals
    //      of the phase before the previous one, then this phase's own stream if it is a
    //      dense group (followed by a grid barrier that keeps a dense stack in model order).
    const int itemsP = (prow + 7) >> 3, itemsO = (orow + 7) >> 3;
    const int padP = ((itemsP + (1 << rpp_log2) - 1) >> rpp_log2) << rpp_log2;
    const int padO = ((itemsO + (1 << rpp_log2) - 1) >> rpp_log2) << rpp_log2;
    const int hold_log2 = q.lpr_log2 - 3;          // lanes per held row after reduce8
    const int lanegroups = kNW << rpp_log2;
#pragma unroll 1
    for (int part = 0; part < 2; ++part) {
      if (part == 1 && (mask_pp || dense)) {
        const int len_pp = plan[t - 2 >= 0 ? t - 2 : 0].len, g_pp = plan[t - 2 >= 0 ? t - 2 : 0].gi0;
#pragma unroll 1
        for (int u = 0; u < 3 && ok; ++u) {
          const PersistGroup* gw = nullptr;
          if (u < 2) {
            if (u < len_pp && (mask_pp & (1u << u))) gw = p.groups + g_pp + u;
          } else if (dense) {
            gw = &g;
          }
          if (!gw) continue;
          if (u < 2) {
            if (tid == 0) {
              grid_wait(gw->bar + 2 + parity, (unsigned)G, p, misc);
              __threadfence();
            }
            csync();
            if (*abort) return;
          }
          const float* src = u < 2 ? gw->r
                                   : gw->x + (long long)slot_io * gw->x_step_stride + (size_t)p.token * gw->d;
          ok = w_stream(p, *gw, src, gw->y + (size_t)p.token * gw->O, u == 2, smem, n, misc);
          if (u == 2) {
            if (tid == 0) {
              red_relaxed_u32(gw->bar + parity, 1u);
              grid_wait(gw->bar + parity, (unsigned)G, p, misc);
              if (cta == 0)
                p.gate_log[((size_t)slot_io * p.log_step_stride + pl.gi) * p.n_tokens + p.token] = 1;
            }
            csync();
          }
        }
        tr.mark(6);
        if (*abort) return;
      }
      if (!gsi) continue;
      const bool image = part == 1;
      const int nchunks = image ? ochunks : pchunks, nrows = image ? orow : prow;
      const int id0 = image ? padP : 0, id1 = image ? padP + padO : padP;
      const unsigned n0 = image ? n : n_p0;
      float* out = image ? g.y + (size_t)p.token * g.O + pl.o0 : g.r + pl.p0;
      if (image) {
        n += ochunks;
        ok = ok && chunks_landed(smem, n0, ochunks, abort);
        tr.mark(7);
      }
      float sr = 0.f;
      int released = 0;
      if (ok) {
        int id = (warp << rpp_log2) + q.sub;
        if (id < id0) id += ((id0 - id + lanegroups - 1) / lanegroups) * lanegroups;
#pragma unroll 1
        for (; __any_sync(0xffffffffu, id < id1); id += lanegroups) {
          const bool live = id < id1;
          const int row0g = live ? (id - id0) << 3 : 0;            // first row, within the slab
          const int ci = min(row0g >> q.rc_log2, nchunks - 1);
          const int ci_warp = __shfl_sync(0xffffffffu, live ? ci : nchunks - 1, 0);  // ids ascend with the lane
          if (lane == 0)
            for (; released < ci_warp; ++released) mbar_arrive(&empty[(n0 + released) % kNB]);
          released = ci_warp;
          const uint4* tile = reinterpret_cast<const uint4*>(ring + s_off[(n0 + ci) % kNB]);
          const int r_lo = ci << q.rc_log2, rows = min(rc, nrows - r_lo);
          const int row0 = row0g - r_lo;
          float v[8];
          dot8(tile, s_c, q, row0, rows, v);
          const float dot = reduce8(v, q.cl, LPR);
          const int row = row0 + (q.cl >> hold_log2);
          if (live && (q.cl & ((1 << hold_log2) - 1)) == 0 && row < rows && row0g < nrows) {
            if (image) {
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
          for (; released < nchunks; ++released) mbar_arrive(&empty[(n0 + released) % kNB]);
      }
      if (!image) {
        sr = warp_sum(sr);
        if (lane == 0) misc->sr[warp] = sr;
      }
      tr.mark(image ? 8 : 5);
    }
    if (!ok && !*abort) fail(p, misc, 8);
    if (*abort) return;

    contrib_p = gsi && prow > 0;
    if (gsi) {
      e_p = x2_own > 0.0 ? exp_above(x2_own) : 0;
      r2word_p = acc + k + 2;
    }
    mask_pp = mask_p;
  }
  if (tid == 0) bulk_reduce_wait_read();
  tr.flush(p);
  // Every CTA read the counters at its start and has since taken part in the
  // last group's exchange, so they may advance now.
  if (cta == 0 && tid == 0 && ok && !*abort) {
    *p.epoch = epoch + 1;
    if (p.use_counter && p.advance) *p.step = step + 1;
  }
}

template <bool kPairs, int kK>
__global__ void __launch_bounds__(kThreadsP, 1) k_decode_step(const __grid_constant__ PersistParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kNB;
  Misc* misc = reinterpret_cast<Misc*>(smem + kOffMisc);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kNB; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kNW);
    }
    misc->abort = 0;
    // shared memory keeps what the previous launch on this SM left: the producer must not
    // mistake an old decision for this launch's
    misc->fire[0] = misc->fire[1] = misc->fire[2] = misc->fire[3] = 0;
    misc->decision[0] = misc->decision[1] = misc->decision[2] = misc->decision[3] = 0u;
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
