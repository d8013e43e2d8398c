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
//   statistics  one warp: max |x| and sum x^2 over this CTA's rows of x (requested and
//               published one row pass ahead: the inputs of a stack are pre-staged); the
//               maximum goes out as a tagged 32-bit word (no fence: the word validates itself)
//   pass 1      partial c = P_slab^T x_slab                              (line 1)
//   exchange    every CTA adds, as 64-bit fixed-point numbers whose upper bits count the
//               arrivals (integer addition is order-free, so the sums are bit-reproducible),
//               its partial c_j (scale from the group's max |x|, collected from the tagged
//               words during pass 1) and its partial ||x||^2 with ONE bulk reduction
//               (cp.reduce.async.bulk), and its partial ||r||^2 of the PREVIOUS phase; one
//               warp then polls the accumulators until all have arrived
// Basis and images are stored as 16 x 16 tiles of four row-major 8 x 8 blocks, so both passes
// and the image rows run on the tensor cores with one ldmatrix per tile (plain: the A operand
// of the row passes; transposed: the B operands of pass 1, which contracts over the tile's
// rows): x and c enter as three bf16 terms each (hi + mid + lo = the fp32 value), so every
// product is exact and the sums are fp32.
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
constexpr int kNB = 64;                     // chunks in flight at most (one barrier pair each)
constexpr int kChunk = 16384;               // largest chunk
static_assert(kPersistMaxWRows <= kPersistConsumerWarps * 32, "one thread per row of a W stream");
constexpr int kWVecMax = 5;                 // 16-byte vectors of a row one lane may own in the W stream (d <= 16384)
constexpr unsigned kLocalSpinLimit = 1u << 20;   // waits inside the CTA (ring, producer hand-off)
constexpr int kCountShift = 54;
constexpr unsigned long long kOne = 1ull << kCountShift;

// What one CTA does in one tick of a launch, worked out once at the start of the launch.
// Rows are dealt in groups of 16 (one tile row).
struct Plan {
  short gi;        // the group whose fast path (or dense stream) this CTA runs in this tick
  short gi0;       // first group of the tick's phase
  unsigned char len, next_len;   // groups in this phase and in the next
  unsigned char kind;            // 0 nothing (closing ticks), 1 gated subspace group, 2 dense group
  unsigned char zeroer;          // this CTA clears the group's counters for the next launch
  short pg, og;                  // 16-row groups of the basis slab and of the image slab
  short pchunks, ochunks;        // ... and their ring chunks
  int p0, o0;                    // first rows
  short lc, n_contrib;           // index within the group's share of the grid; CTAs that own basis rows
  short gc_log2, pad;            // log2 of the 16-row groups per 16 KB chunk
};
static_assert(sizeof(Plan) == 32, "one plan record");

// Groups [a, b) of n that part i of `parts` owns: an even split, or one group each for the
// first n parts when there are fewer groups than parts.
__device__ __forceinline__ void deal(int n, int parts, int i, int& a, int& b) {
  if (n >= parts) {   // i <= parts <= 256 and n < 2^20: the products fit 32 bits
    a = (int)((unsigned)i * (unsigned)n / (unsigned)parts);
    b = (int)((unsigned)(i + 1) * (unsigned)n / (unsigned)parts);
  } else {
    a = min(i, n);
    b = min(i + 1, n);
  }
}

// shared memory map (bytes)
constexpr int kOffBar = 0;          // full[kNB], empty[kNB]
constexpr int kOffLin = 1024;       // producer: ring position (bytes placed before it) of every chunk in flight (kNB words)
constexpr int kOffOff = 1280;       // offset of every chunk in flight within the ring (kNB words), for the consumers
constexpr int kOffMisc = 1536;      // scalars
constexpr int kOffTrace = 1792;     // cycle counters of the trace (16 words)
constexpr int kOffProd = 1920;      // state of the producer thread (16 bytes)
constexpr int kOffX = 2048;         // x of this CTA's basis rows, two buffers (kPersistMaxPRows floats each)
constexpr int kOffXt = kOffX + 3 * kPersistMaxPRows * 4;  // ... as three bf16 terms in A-operand order, two buffers (16 tile rows x 256 B each)
constexpr int kOffCb = kOffXt + 2 * 4096;                 // c as three bf16 terms in B-operand order (32 tile columns x 256 B)
constexpr int kOffFx = kOffCb + 8192;                     // fixed-point partial c and ||x||^2, source of the bulk reduction (514 words)
constexpr int kOffPlan = kOffFx + 4224;                   // the launch's plan (kPersistMaxTicks records)
constexpr int kOffDesc = kOffPlan + kPersistMaxTicks * 32;   // 8 group descriptors, 256 B each
constexpr int kDescSlots = 16;
constexpr int kOffYacc = kOffDesc + kDescSlots * 512;     // W stream: per-warp partial results (kNW x kPersistMaxWRows floats)
constexpr int kOffRing = ((kOffYacc + kNW * kPersistMaxWRows * 4 + 1023) / 1024) * 1024;
constexpr int kRingBytes = (232448 - kOffRing) / 1024 * 1024;
constexpr int kSmemBytes = kOffRing + kRingBytes;
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 CTA");
static_assert(kOffXt % 16 == 0 && kOffCb % 16 == 0 && kOffFx % 16 == 0 && kOffPlan % 16 == 0 && kOffDesc % 16 == 0, "alignment");
static_assert(sizeof(PersistGroup) <= 512 && sizeof(PersistGroup) % 4 == 0, "descriptor slot");
constexpr int kDescWords = (int)(sizeof(PersistGroup) / 4);

struct Misc {
  int abort;
  unsigned amax_bits[2];    // by tick parity: max |x| of the phase's group (>= 0x7f800000: a non-finite token)
  float x2_part[2];         // this CTA's sum of x^2 over its rows, by tick parity
  int fire[4];              // decisions on the previous phase's groups, by tick parity: 1 = stream W
  double x2;                // ||x||^2 of this phase's group
  unsigned long long r2_acc;   // this CTA's ||r||^2 of the tick's phase in fixed point; the upper bits count the warps
  volatile unsigned decision[4];   // hand-off to the producer: (phase + 1) << 8 | fire mask
  volatile int stop[2];     // the abort flag as thread 0 saw it before a barrier (one word per barrier of the tick, so that
                            // a warp still reading one cannot see the next write): every warp leaves at the same barrier
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
__device__ __forceinline__ void mbar_arrive_n(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
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
// Before a thread that issued bulk reductions or asynchronous copies leaves the kernel: all of
// them complete (a CTA must not retire with such operations in flight).
__device__ __forceinline__ void async_drain() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  asm volatile("cp.async.wait_all;" ::: "memory");
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
__device__ __noinline__ void fail_at(int* status, Misc* misc, int site) {
  misc->abort = 1;
  atomicExch(status, (int)GSI_ERR_TIMEOUT);
  atomicCAS(status + 1, 0, site);
}
__device__ __forceinline__ void fail(const PersistParams& p, Misc* misc, int site) { fail_at(p.status, misc, site); }

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

// ------------------------------------------------------------------ the ring
// Chunks of any size up to 16 KB are packed back to back in a circular byte buffer (a chunk
// never wraps: the tail of the buffer is skipped instead).  `lin` counts bytes placed so far,
// skipped tails included, so lin % kRingBytes is the physical offset; chunk n uses barrier
// pair n % kNB.  The producer publishes the offset of chunk n in s_off[n % kNB] before it arms
// the chunk's "full" barrier; producer and consumers walk the same sequence of chunks, so a
// consumer needs only the sequence number.
struct Producer {      // state of the producer thread, kept in shared memory
  unsigned n;          // sequence number of the next chunk
  unsigned lin;        // bytes placed so far
  unsigned tail_n;     // oldest chunk not yet given back by the consumers
  unsigned tail_lin;   // where it starts
};

// Reserve `bytes` for chunk n: waits (bounded) until the consumers have given back every
// older chunk that still overlaps the place, and a barrier pair is free.  Returns the
// offset, or 0xffffffff when a wait gave up.  Out of line: one copy for every kind of chunk.
__device__ __noinline__ unsigned producer_acquire(unsigned char* smem, unsigned bytes) {
  Producer& pr = *reinterpret_cast<Producer*>(smem + kOffProd);
  uint64_t* empty = reinterpret_cast<uint64_t*>(smem + kOffBar) + kNB;
  unsigned* s_lin = reinterpret_cast<unsigned*>(smem + kOffLin);
  unsigned* s_off = reinterpret_cast<unsigned*>(smem + kOffOff);
  volatile int* abort = &reinterpret_cast<Misc*>(smem + kOffMisc)->abort;
  unsigned n = pr.n, lin = pr.lin, tail_n = pr.tail_n, tail_lin = pr.tail_lin;
  unsigned off = lin % (unsigned)kRingBytes;
  if (off + bytes > (unsigned)kRingBytes) {
    lin += (unsigned)kRingBytes - off;
    off = 0;
  }
  const unsigned start = lin;
  lin += bytes;
  while (n - tail_n >= (unsigned)kNB || (tail_n < n && lin - tail_lin > (unsigned)kRingBytes)) {
    if (!mbar_wait(&empty[tail_n % kNB], (tail_n / kNB) & 1u, abort)) return 0xffffffffu;
    ++tail_n;
    tail_lin = tail_n < n ? s_lin[tail_n % kNB] : start;
  }
  if (tail_n == n) tail_lin = start;
  s_lin[n % kNB] = start;
  s_off[n % kNB] = off;
  pr.lin = lin;
  pr.tail_n = tail_n;
  pr.tail_lin = tail_lin;
  return off;
}

// The W stream of one group for this CTA: its w_rows[j] consecutive rows of every map j are
// one contiguous run of memory, copied as contiguous pieces of w_pr whole rows (at most 32 KB:
// large contiguous copies are what reaches the memory system's bandwidth).
__device__ __forceinline__ bool produce_w(const PersistGroup& g, unsigned char* smem) {
  Producer& prs = *reinterpret_cast<Producer*>(smem + kOffProd);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kNB;
  unsigned* s_lin = reinterpret_cast<unsigned*>(smem + kOffLin);
  unsigned* s_off = reinterpret_cast<unsigned*>(smem + kOffOff);
  unsigned char* base = smem + kOffRing;
  volatile int* abort = &reinterpret_cast<Misc*>(smem + kOffMisc)->abort;
  // the ring state in registers for the length of the stream (thousands of pieces, one every
  // few hundred cycles: the out-of-line acquire with its state in shared memory is too slow)
  unsigned n = prs.n, lin = prs.lin, tail_n = prs.tail_n, tail_lin = prs.tail_lin;
  bool ok = true;
  const int cta = blockIdx.x;
  const int d = g.d, pr = g.w_pr;
  for (int j = 0; j < g.n_maps && ok; ++j) {
    const int dout = g.off[j + 1] - g.off[j], rows = g.w_rows[j];
    const int row0 = cta * rows;
    const int live = min(rows, dout - row0);
    for (int r0 = 0; r0 < live; r0 += pr) {
      const uint32_t bytes = (uint32_t)min(pr, live - r0) * d * 2;
      unsigned off = lin % (unsigned)kRingBytes;
      if (off + bytes > (unsigned)kRingBytes) {
        lin += (unsigned)kRingBytes - off;
        off = 0;
      }
      const unsigned start = lin;
      lin += bytes;
      while (n - tail_n >= (unsigned)kNB || (tail_n < n && lin - tail_lin > (unsigned)kRingBytes)) {
        if (!mbar_wait(&empty[tail_n % kNB], (tail_n / kNB) & 1u, abort)) {
          ok = false;
          break;
        }
        ++tail_n;
        tail_lin = tail_n < n ? s_lin[tail_n % kNB] : start;
      }
      if (!ok) break;
      if (tail_n == n) tail_lin = start;
      s_lin[n % kNB] = start;
      s_off[n % kNB] = off;
      uint64_t* fb = &full[n % kNB];
      mbar_expect_tx(fb, bytes);
      bulk_g2s(base + off, g.W[j] + (size_t)(row0 + r0) * d, bytes, fb);
      ++n;
    }
  }
  prs.n = n;
  prs.lin = lin;
  prs.tail_n = tail_n;
  prs.tail_lin = tail_lin;
  return ok;
}

// Tile rows [a, b) (16 matrix rows each, row_bytes bytes) of a tiled matrix of rank k as chunks
// of whole tile rows (as many per chunk as 16 KB hold of the bf16 form).
__device__ __forceinline__ bool produce_rows(const void* base, int k, int row_bytes, int a, int b,
                                             unsigned char* smem) {
  Producer& pr = *reinterpret_cast<Producer*>(smem + kOffProd);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  const int gc = kChunk / (k * 32);
  for (int r = a; r < b; r += gc) {
    const int groups = min(gc, b - r);
    const uint32_t bytes = (uint32_t)(groups * row_bytes);
    const unsigned off = producer_acquire(smem, bytes);
    if (off == 0xffffffffu) return false;
    uint64_t* fb = &full[pr.n % kNB];
    mbar_expect_tx(fb, bytes);
    bulk_g2s(smem + kOffRing + off, static_cast<const char*>(base) + (size_t)r * row_bytes, bytes, fb);
    ++pr.n;
  }
  return true;
}

__device__ void producer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  Producer& pr = *reinterpret_cast<Producer*>(smem + kOffProd);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  pr.n = 0;
  pr.lin = 0;
  pr.tail_n = 0;
  pr.tail_lin = 0;
  volatile int* abort = &misc->abort;
  bool ok = true;
  // ticks: tick t runs the rows of phase t, pass 1 of phase t + 1 and the gated residuals of
  // phase t - 2; the work of a tick, in ring order (the order in which the consumers give the
  // chunks back): the basis slab of phase t + 1 for pass 1 (that of the first phase comes before
  // the first tick), the basis slab of phase t again for its residual rows, the image slab of
  // phase t, the W pieces of the gated groups (or of a dense group)
  const Plan* plan = reinterpret_cast<const Plan*>(smem + kOffPlan);
  const int n_ticks = p.n_phases + 2;
  if (plan[0].kind == 1) {
    const PersistGroup* g0 = p.groups + plan[0].gi;
    ok = produce_rows(g0->P, g0->k, g0->k * 32, plan[0].p0 >> 4, (plan[0].p0 >> 4) + plan[0].pg, smem);
  }
#pragma unroll 1
  for (int t = 0; t < n_ticks && ok; ++t) {
    const Plan& pl = plan[t];
    const PersistGroup* g = p.groups + pl.gi;   // read only when the tick has a group
    if (t + 1 < p.n_phases && plan[t + 1].kind == 1) {
      const Plan& pn = plan[t + 1];
      const PersistGroup* gn = p.groups + pn.gi;
      ok = produce_rows(gn->P, gn->k, gn->k * 32, pn.p0 >> 4, (pn.p0 >> 4) + pn.pg, smem);
    }
    if (ok && pl.kind == 1) {
      ok = produce_rows(g->P, g->k, g->k * 32, pl.p0 >> 4, (pl.p0 >> 4) + pl.pg, smem);   // once more, for the residual rows
      if (ok)
        ok = produce_rows(g->WP, g->k, persist_image_row_bytes(g->k, g->flags & GSI_FLAG_FP8_IMAGE), pl.o0 >> 4,
                          (pl.o0 >> 4) + pl.og, smem);
    }
    unsigned wmask = 0;
    const int len_pp = t >= 2 ? plan[t - 2].len : 0, g_pp = t >= 2 ? plan[t - 2].gi0 : 0;
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
    if (wmask || pl.kind == 2) {
#pragma unroll 1
      for (int u = 0; ok && u < 3; ++u) {
        const PersistGroup* gw = nullptr;
        if (u < 2) {
          if (u < len_pp && (wmask & (1u << u))) gw = &p.groups[g_pp + u];
        } else if (pl.kind == 2) {
          gw = g;
        }
        if (gw) ok = produce_w(*gw, smem);
      }
    }
  }
  if (!ok && !*abort) fail(p, misc, 1);
  // Every copy issued must have landed before the CTA may give up its shared
  // memory: wait (bounded) for the last kNB chunks.
  {
    const unsigned first = pr.n > (unsigned)kNB ? pr.n - kNB : 0;
    for (unsigned c = first; c < pr.n; ++c) {
      const unsigned slot = c % kNB, ph = (c / kNB) & 1u;
      for (unsigned it = 0; it < kLocalSpinLimit; ++it)
        if (mbar_try(&full[slot], ph)) break;
    }
  }
}

// ------------------------------------------------------------------ consumer
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

// Two E4M3 codes -> two bf16 (exact: every E4M3 value is a bf16 value), low byte to low half.
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t two) {
  uint32_t h, out;
  unsigned short lo16, hi16;
  float lo, hi;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"((unsigned short)two));
  asm("mov.b32 {%0, %1}, %2;" : "=h"(lo16), "=h"(hi16) : "r"(h));
  asm("cvt.f32.f16 %0, %1;" : "=f"(lo) : "h"(lo16));
  asm("cvt.f32.f16 %0, %1;" : "=f"(hi) : "h"(hi16));
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out) : "f"(hi), "f"(lo));
  return out;
}

// D (16 x 8, fp32) += A (16 x 16, bf16) B (16 x 8, bf16) on the tensor cores.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
// One 16 x 16 bf16 tile (512 bytes: its four 8 x 8 blocks one after the other, each row-major
// with 16-byte rows; block order (rows 0-7, columns 0-7), (8-15, 0-7), (0-7, 8-15), (8-15, 8-15))
// from shared memory; `lane_row` = the tile's base + 16 * lane.  Plain: the A operand of
// mma.m16n8k16 over the tile.  Transposed: every block transposed, i.e. the tile as the B
// operands of two instructions that contract over the tile's ROWS (x, y for columns 0-7;
// z, w for columns 8-15).
__device__ __forceinline__ uint4 ldsm_tile(const void* lane_row) {
  uint4 r;
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "r"(smem_u32(lane_row)));
  return r;
}
__device__ __forceinline__ uint4 ldsm_tile_trans(const void* lane_row) {
  uint4 r;
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "r"(smem_u32(lane_row)));
  return r;
}
// Arrivals that the unit `j` of `u` units sharing a chunk owes the chunk's "empty" barrier
// (which expects kNW): the shares of a chunk's units add up to kNW.
__device__ __forceinline__ uint32_t unit_share(int j, int u) {
  return (uint32_t)(kNW / u + (j < kNW % u ? 1 : 0));
}
// v = hi + mid + lo, each a bf16 (round to nearest; the remainders are exact in fp32).
__device__ __forceinline__ void split3(float v, unsigned short (&t)[3]) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(h);
  const __nv_bfloat16 m = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(m);
  const __nv_bfloat16 l = __float2bfloat16_rn(r2);
  t[0] = __bfloat16_as_ushort(h);
  t[1] = __bfloat16_as_ushort(m);
  t[2] = __bfloat16_as_ushort(l);
}
// Element e (0..15) of vector chunk `blk` as term g of a three-term operand: index of its
// 16-bit slot in an array of 256-byte blocks laid out one 8-byte word per lane (the A operand
// rows 0..2 of mma.m16n8k16, or its B operand columns 0..2: lane = 4 g + (e % 8) / 2, word half
// e / 8, element e % 2).
__device__ __forceinline__ int term_slot(int blk, int e, int g) {
  return (((blk * 32 + g * 4 + ((e & 7) >> 1)) * 2 + (e >> 3)) * 2) + (e & 1);
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

// One piece of the W stream for one warp: rows_p rows of rvec vectors; this lane owns vectors
// lane + 32 i (i < VPL) of the warp's range (first = pointer to its first vector of row 0,
// nvalid = how many of its VPL vectors exist); `in` holds its share of the input.  RPI rows at
// a time (2 or 1: more rows in flight cost registers that the tick loop around the stream
// needs); two rows share five shuffles (the first level sends half of the values to the
// partner).  Results to part[row].
// The piece goes back to the producer (release_n arrivals on `eb`) as soon as its last rows
// are in registers, before the sums over the lanes: the arrival is predicated on a value that
// every load of the warp feeds (a comparison that never fails), so it cannot be issued before
// those loads have returned.
template <int VPL, int RPI>
__device__ __forceinline__ void w_piece(const uint4* first, int rvec, int rows_p, int nvalid,
                                        const unsigned long long (&in)[kWVecMax][4], float* part,
                                        uint64_t* eb, uint32_t release_n) {
  const int lane = threadIdx.x & 31;
  constexpr unsigned kNever = 0x7fc5a5a5u;   // a NaN pattern no arithmetic instruction produces
#pragma unroll 1
  for (int ra = 0; ra < rows_p; ra += RPI) {
    unsigned long long a[RPI], b[RPI];   // two chains of dependent additions per row
#pragma unroll
    for (int q = 0; q < RPI; ++q) a[q] = b[q] = 0ull;
    uint4 w[VPL][RPI];
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int q = 0; q < RPI; ++q) {
        // rows past the piece read the last row again (dropped below); vectors past the row's
        // end are not read at all
        w[i][q] = make_uint4(0u, 0u, 0u, 0u);
        if (i < nvalid) w[i][q] = first[(size_t)min(ra + q, rows_p - 1) * rvec + 32 * i];
      }
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int q = 0; q < RPI; ++q) {
        fma2(a[q], bf16x2_to_f32x2(w[i][q].x), in[i][0]);
        fma2(b[q], bf16x2_to_f32x2(w[i][q].y), in[i][1]);
        fma2(a[q], bf16x2_to_f32x2(w[i][q].z), in[i][2]);
        fma2(b[q], bf16x2_to_f32x2(w[i][q].w), in[i][3]);
      }
    float v[RPI];
#pragma unroll
    for (int q = 0; q < RPI; ++q) v[q] = sum2(a[q]) + sum2(b[q]);
    const bool last = ra + RPI >= rows_p;
    float v0 = v[0];
    int q_mine = 0, keep = 31;   // the row this lane ends up with, and which lanes write (lane & keep == 0)
    if constexpr (RPI == 2) {
      const bool up = lane & 16;
      const float s0 = up ? v[0] : v[1];
      const float r0v = __shfl_xor_sync(0xffffffffu, s0, 16);
      v0 = (up ? v[1] : v[0]) + r0v;
      q_mine = lane >> 4;
      keep = 15;
    }
    // v0 now depends on every row loaded above
    if (last) {
      __syncwarp();
      if (lane == 0 && __float_as_uint(v0) != kNever) mbar_arrive_n(eb, release_n);
    }
    if constexpr (RPI == 1) v0 += __shfl_xor_sync(0xffffffffu, v0, 16);
    v0 += __shfl_xor_sync(0xffffffffu, v0, 8);
    v0 += __shfl_xor_sync(0xffffffffu, v0, 4);
    v0 += __shfl_xor_sync(0xffffffffu, v0, 2);
    v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
    if ((lane & keep) == 0 && ra + q_mine < rows_p) part[ra + q_mine] = v0;
  }
}

// ---- W stream: y_rows (+)= W_rows . src (src = r of a gated group, or x for the dense
// baseline), pieces of whole rows taken from the ring in the producer's order.  The consumer
// warps form teams of nw warps; a team takes every T-th piece, so T pieces are worked on at
// once and the latency of one piece (wait, loads, sums over the lanes) is hidden by the
// others.  Within a team every warp owns a range of columns and keeps its share of src in
// registers for the whole stream (four or five 16-byte vectors of W per lane and row; no
// staging in shared memory).  The partial sums of a row meet in shared memory and are added
// in warp order at the end (reproducible).  `n` is the consumers' chunk sequence number on
// entry, the return value the one after the stream; a wait that gave up sets the abort flag.
// Inlined at its two call sites (an out-of-line call makes the tick loop keep its state in
// local memory); both sit where little of the tick's state is alive.
// How the consumer warps share a W stream of input width d.
struct WGeo {
  int d, pr, n_maps, rvec, vpl, nw, T, team, wi, v_lo, v_hi, nvalid;
  bool active;
  uint32_t release_n;
};
__device__ __forceinline__ WGeo w_geometry(const PersistGroup* gp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  WGeo q;
  q.d = gp->d;
  q.pr = gp->w_pr;
  q.n_maps = gp->n_maps;
  q.rvec = q.d >> 3;                                         // 16-byte vectors per row
  q.vpl = q.rvec > 4 * kNC ? 5 : 4;
  q.nw = (q.rvec + 32 * q.vpl - 1) / (32 * q.vpl);           // warps of a team
  q.T = kNW / q.nw;                                          // teams
  q.team = warp / q.nw;
  q.wi = warp - q.team * q.nw;
  q.active = q.team < q.T;
  q.v_lo = min(q.rvec, q.wi * 32 * q.vpl);                   // this warp's vectors of every row
  q.v_hi = min(q.rvec, q.v_lo + 32 * q.vpl);
  q.nvalid = (q.v_hi - q.v_lo - lane + 31) >> 5;             // how many of this lane's vectors exist
  q.release_n = q.wi == 0 ? (uint32_t)(kNW - q.nw + 1) : 1u; // a team's first warp also arrives for all other warps
  return q;
}
// This lane's share of the input: vectors v_lo + lane + 32 i.
__device__ __forceinline__ void w_load_in(const WGeo& q, const float* src, unsigned long long (&in)[kWVecMax][4]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int i = 0; i < kWVecMax; ++i) {
    const int v = q.v_lo + lane + 32 * i;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (q.active && v < q.v_hi) {
      a = __ldcg(reinterpret_cast<const float4*>(src) + 2 * v);
      b = __ldcg(reinterpret_cast<const float4*>(src) + 2 * v + 1);
    }
    in[i][0] = pack2(a.x, a.y);
    in[i][1] = pack2(a.z, a.w);
    in[i][2] = pack2(b.x, b.y);
    in[i][3] = pack2(b.z, b.w);
  }
}

__device__ __forceinline__ unsigned w_run(const PersistGroup* gp, const WGeo& q,
                                          const unsigned long long (&in)[kWVecMax][4], float* y, bool dense,
                                          unsigned char* smem, unsigned n, int* status, bool traced) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kNB;
  const unsigned* s_off = reinterpret_cast<const unsigned*>(smem + kOffOff);
  unsigned char* ring = smem + kOffRing;
  float* s_part = reinterpret_cast<float*>(smem + kOffYacc);
  Misc* misc = reinterpret_cast<Misc*>(smem + kOffMisc);
  volatile int* abort = &misc->abort;
  const int tid = threadIdx.x, lane = tid & 31;
  const int cta = blockIdx.x;
  Trace tr;
  tr.acc = (traced && tid == 0) ? reinterpret_cast<unsigned long long*>(smem + kOffTrace) : nullptr;
  tr.t = clock64();
  const int pr = q.pr, n_maps = q.n_maps, rvec = q.rvec, nw = q.nw, T = q.T, team = q.team, wi = q.wi;
  const bool active = q.active;
  bool ok = true;
  // thread i owns row i of this CTA's rows (all maps, in order): its y so far (the image row,
  // written by another CTA and visible by now) is fetched while the stream runs
  float* yp = nullptr;
  float yold = 0.f;
  {
    int yb = 0;
#pragma unroll 1
    for (int j = 0; j < n_maps; ++j) {
      const int dout = gp->off[j + 1] - gp->off[j], rows = gp->w_rows[j];
      const int live = max(min(rows, dout - cta * rows), 0);
      if (tid >= yb && tid < yb + live) yp = y + gp->off[j] + cta * rows + (tid - yb);
      yb += live;
    }
    if (yp && !dense) yold = __ldcg(yp);
  }
  int ybase = 0, pi = 0;   // rows of the maps before this one; pieces of this stream so far
  tr.mark(10);
#pragma unroll 1
  for (int j = 0; j < n_maps; ++j) {
    const int dout = gp->off[j + 1] - gp->off[j], rows = gp->w_rows[j];
    const int live = min(rows, dout - cta * rows);
#pragma unroll 1
    for (int r0 = 0; r0 < live; r0 += pr, ++pi) {
      const int rows_p = min(pr, live - r0);
      const unsigned slot = n % kNB, ph = (n / kNB) & 1u;
      ++n;
      if (!active || pi % T != team) continue;
      if (ok && !__all_sync(0xffffffffu, mbar_wait(&full[slot], ph, abort))) ok = false;   // (for the warp as a whole)
      tr.mark(11);
      if (ok) {
        const uint4* piece = reinterpret_cast<const uint4*>(ring + s_off[slot]) + q.v_lo + lane;
        float* part = s_part + wi * kPersistMaxWRows + ybase + r0;
        uint64_t* eb = &empty[slot];
        if (q.vpl == 5) w_piece<5, 1>(piece, rvec, rows_p, q.nvalid, in, part, eb, q.release_n);
        else if (pr >= 2) w_piece<4, 2>(piece, rvec, rows_p, q.nvalid, in, part, eb, q.release_n);
        else w_piece<4, 1>(piece, rvec, rows_p, q.nvalid, in, part, eb, q.release_n);
      }
      tr.mark(12);
    }
    ybase += max(live, 0);
  }
  if (!ok && !*abort) fail_at(status, misc, 3);
  csync();
  // rows back to y: the warps' partial sums in warp order, onto the value fetched at the start
  if (ok && yp) {
    float acc = 0.f;
#pragma unroll 1
    for (int q = 0; q < nw; ++q) acc += s_part[q * kPersistMaxWRows + tid];
    *yp = yold + acc;
  }
  csync();   // the partial sums may be overwritten by the next stream
  tr.mark(13);
  return n;
}


// Geometry, input share and stream in one go.
__device__ __forceinline__ unsigned w_stream(const PersistGroup* gp, const float* src, float* y, bool dense,
                                             unsigned char* smem, unsigned n, int* status, bool traced) {
  const WGeo q = w_geometry(gp);
  unsigned long long in[kWVecMax][4];
  w_load_in(q, src, in);
  return w_run(gp, q, in, y, dense, smem, n, status, traced);
}

// The statistics warp: the group's max |x| for tick `tt` from the tagged words of all
// contributing CTAs (lane l owns words l, l+32, ...).  `first` holds a first round of loads
// issued earlier (split phase: they flew while the warp did other work); further rounds are
// polled here.  Out of line.
constexpr int kXmaxWords = (kPersistMaxGrid + 31) / 32;
__device__ __forceinline__ void xmax_issue(const unsigned* xmax, int n_contrib, unsigned (&w)[kXmaxWords]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int i = 0; i < kXmaxWords; ++i) {
    const int w_i = lane + 32 * i;
    w[i] = w_i < n_contrib ? ld_relaxed_u32(xmax + w_i) : 0xffffffffu;   // all loads in flight together
  }
}
__device__ __noinline__ void xmax_collect(unsigned char* smem, int tt, unsigned tag, unsigned spin_limit,
                                          int* status, unsigned w0, unsigned w1, unsigned w2,
                                          unsigned w3, unsigned w4) {
  static_assert(kXmaxWords == 5, "argument list");
  const Plan& pn = reinterpret_cast<const Plan*>(smem + kOffPlan)[tt];
  Misc* misc = reinterpret_cast<Misc*>(smem + kOffMisc);
  const PersistGroup& gn =
      *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (pn.gi & (kDescSlots - 1)) * 512);
  const int lane = threadIdx.x & 31;
  unsigned w[kXmaxWords] = {w0, w1, w2, w3, w4};
  unsigned m = 0, it = 0;
  for (;;) {
    bool all = true;
    m = 0;
#pragma unroll
    for (int i = 0; i < kXmaxWords; ++i) {
      if (lane + 32 * i < pn.n_contrib) {
        all = all && ((w[i] >> 31) == tag);
        m = max(m, w[i] & 0x7fffffffu);
      }
    }
    if (__all_sync(0xffffffffu, all)) break;
    if (++it > spin_limit || ((it & 1023u) == 0 && misc->abort)) {
      if (!misc->abort && lane == 0) fail_at(status, misc, 4);
      break;
    }
    xmax_issue(gn.xmax, pn.n_contrib, w);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) misc->amax_bits[tt & 1] = m;
}

// The statistics warp, for tick `tt`: (request = true) ask for this CTA's rows of x into buffer
// tt & 1; (request = false) wait for them, take max |x| and sum x^2 over them, publish the
// maximum at once as a tagged word, keep the sum for the tick's exchange, and leave x as three
// bf16 terms in the operand order of pass 1.  Out of line: two call sites, one copy.
__device__ __noinline__ void stat_warp_step(unsigned char* smem, int tt, bool request, int slot_io, int token,
                                            unsigned tag) {
  const Plan& pn = reinterpret_cast<const Plan*>(smem + kOffPlan)[tt];
  if (pn.kind != 1) return;
  const int lane = threadIdx.x & 31;
  const PersistGroup& gn =
      *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (pn.gi & (kDescSlots - 1)) * 512);
  float* sx = reinterpret_cast<float*>(smem + kOffX) + (tt % 3) * kPersistMaxPRows;
  const int rows = pn.pg * 16;
  if (request) {
    const float* src = gn.x + (long long)slot_io * gn.x_step_stride + (size_t)token * gn.d + pn.p0;
    const int live = min(rows, gn.d - pn.p0);   // rows past d belong to the zero padding of P
#pragma unroll 1
    for (int i = lane; i < rows; i += 32) {
      if (i < live)
        cp_async4(sx + i, src + i);
      else
        sx[i] = 0.f;
    }
    cp_async_commit();
    return;
  }
  cp_async_wait_all();
  __syncwarp();
  unsigned short* xt = reinterpret_cast<unsigned short*>(smem + kOffXt) + (tt & 1) * 2048;
  Misc* misc = reinterpret_cast<Misc*>(smem + kOffMisc);
  float amax = 0.f, s2 = 0.f;
#pragma unroll 1
  for (int i = lane; i < rows; i += 32) {
    const float v = sx[i];
    amax = fmaxf(amax, fabsf(v));
    s2 = fmaf(v, v, s2);
    unsigned short tm[3];
    split3(v, tm);
    const int slot = term_slot(i >> 4, i & 15, 0);
    xt[slot] = tm[0];
    xt[slot + 16] = tm[1];   // the next term is the next row of the operand: four lanes on
    xt[slot + 32] = tm[2];
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
    if (pn.pg > 0) st_relaxed_u32(gn.xmax + pn.lc, bits | (tag << 31));
    misc->x2_part[tt & 1] = s2;
  }
}

// The plan of this launch for this CTA, one thread per tick (all threads of the CTA, before
// the producer and the consumers part).
template <bool kPairs, int kK>
__device__ __forceinline__ void make_plan(const PersistParams& p, unsigned char* smem) {
  Plan* plan = reinterpret_cast<Plan*>(smem + kOffPlan);
  const int cta = blockIdx.x, n_ticks = p.n_phases + 2;
#pragma unroll 1
  for (int t = threadIdx.x; t < n_ticks; t += kThreadsP) {
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
        const int k = kK ? kK : __ldg(&g->k);
        const int gcl = 31 - __clz(kChunk / (k * 32));
        const int gc = 1 << gcl;
        int a, b;
        deal((__ldg(&g->d) + 15) >> 4, ncta, lc, a, b);
        pl.p0 = a * 16;
        pl.pg = (short)(b - a);
        pl.pchunks = (short)((b - a + gc - 1) >> gcl);
        deal((__ldg(&g->O) + 15) >> 4, ncta, lc, a, b);
        pl.o0 = a * 16;
        pl.og = (short)(b - a);
        pl.ochunks = (short)((b - a + gc - 1) >> gcl);
        pl.n_contrib = (short)__ldg(&g->n_contrib);
        pl.gc_log2 = (short)gcl;
      }
    }
    plan[t] = pl;
  }
}

// kPairs = false compiles the pair logic out: stacks without concurrent groups run a smaller
// loop (the per-phase code has to stay short: it is executed once per phase, straight through,
// so its length is paid in instruction fetches).  kK != 0 is a build for stacks whose groups all
// have rank kK (shifts, strides and loop bounds become constants); kK = 0 reads the rank from
// the descriptor.
template <bool kPairs, int kK>
__device__ void consumer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  uint64_t* full_b = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full_b + kNB;
  const unsigned* s_off = reinterpret_cast<const unsigned*>(smem + kOffOff);
  unsigned char* ring = smem + kOffRing;
  float* s_xb = reinterpret_cast<float*>(smem + kOffX);
  unsigned short* s_xt = reinterpret_cast<unsigned short*>(smem + kOffXt);
  unsigned short* s_cb = reinterpret_cast<unsigned short*>(smem + kOffCb);
  unsigned long long* s_fx = reinterpret_cast<unsigned long long*>(smem + kOffFx);
  Plan* plan = reinterpret_cast<Plan*>(smem + kOffPlan);
  volatile int* abort = &misc->abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int lg = lane >> 2, lt = lane & 3;   // row and column pair of this lane in a tensor-core operand
  constexpr int kStatWarp = kNW - 1;   // statistics of x and the collection of max|x|
  constexpr int kP1First = 5;          // warps 0..4 wait for the exchange of the tick's phase ...
  constexpr int kP1 = kStatWarp - kP1First;   // ... while warps 5..13 run pass 1 of the phase after it

  unsigned n = 0;   // chunk sequence number: advances exactly as in producer()
  const int step = p.use_counter ? *p.step : 0;
  const int slot_io = step % p.n_steps;
  const int epoch = *p.epoch;
  const unsigned parity = (unsigned)epoch & 1u, tag = ((unsigned)epoch + 1u) & 1u;
  const int n_ticks = p.n_phases + 2;
  Trace tr;
  tr.start(p, smem);

  auto desc = [&](int i) -> const PersistGroup& {
    return *reinterpret_cast<const PersistGroup*>(smem + kOffDesc + (i & (kDescSlots - 1)) * 512);
  };
  // groups [g0, g0 + cnt) from the device table into their slots (threads 0 .. cnt*kDescWords-1)
  auto desc_load = [&](int g0, int cnt) -> uint32_t {
    return tid < cnt * kDescWords ? __ldg(reinterpret_cast<const uint32_t*>(p.groups + g0) + tid) : 0u;
  };
  auto desc_store = [&](int g0, int cnt, uint32_t w) {
    if (tid < cnt * kDescWords) {
      const int j = tid / kDescWords;
      reinterpret_cast<uint32_t*>(smem + kOffDesc + ((g0 + j) & (kDescSlots - 1)) * 512)[tid - j * kDescWords] = w;
    }
  };
  // the operand rows / columns beyond the three terms stay zero for the whole launch
  for (int i = tid; i < (2 * 4096 + 8192) / 4; i += kNC) reinterpret_cast<uint32_t*>(smem + kOffXt)[i] = 0u;
  // the descriptors of the first two phases (descriptors are staged three phases ahead; the
  // tick before the first phase stages the third)
  {
    const int cnt = plan[0].len + (p.n_phases > 1 ? plan[1].len : 0);
    desc_store(0, cnt, desc_load(0, cnt));
  }
  csync();
  if (warp == kStatWarp) {   // the first phase's rows of x: nothing ran ahead of them
    stat_warp_step(smem, 0, true, slot_io, p.token, tag);
    stat_warp_step(smem, 0, false, slot_io, p.token, tag);
    if (plan[0].kind == 1) {
      unsigned xw[kXmaxWords];
      xmax_issue(desc(plan[0].gi).xmax, plan[0].n_contrib, xw);
      xmax_collect(smem, 0, tag, p.spin_limit, p.status, xw[0], xw[1], xw[2], xw[3], xw[4]);
    }
  }

  unsigned mask_pp = 0;          // gates that fired in the phase before the previous one
  bool ok = true;

#pragma unroll 1
  // Tick t runs the rows of phase t (whose exchange was sent during tick t - 1) and, beside
  // the wait for that exchange, pass 1 and the send of phase t + 1; tick -1 has only the latter.
  for (int t = -1; t < n_ticks; ++t) {   // (a warp whose wait gave up stays in step: the CTA leaves together)
    const Plan pl = t >= 0 ? plan[t] : Plan{};
    const Plan pf = t + 1 < p.n_phases ? plan[t + 1] : Plan{};   // the phase whose pass 1 runs in this tick
    const bool gsi = pl.kind == 1, dense = pl.kind == 2, gsi_f = pf.kind == 1;
    const PersistGroup& g = desc(pl.gi);        // read only when the tick has a group
    const int k = gsi ? (kK ? kK : g.k) : 0;
    const int KT = k >> 4;                      // tile columns
    const int pg = pl.pg, og = pl.og, pchunks = pl.pchunks, ochunks = pl.ochunks, gcl = pl.gc_log2;
    const int n_contrib = pl.n_contrib, lc = pl.lc;
    const int len_p = t >= 1 ? plan[t - 1].len : 0, g_p = t >= 1 ? plan[t - 1].gi0 : 0;
    const float* s_x = s_xb + ((t + 3) % 3) * kPersistMaxPRows;
    unsigned long long* acc = gsi ? g.acc + (size_t)parity * (k + 4) : nullptr;
    const int tp = (t & 1) * 2;

    // the descriptors of the phase three ahead: requested now, stored before the barrier that ends the exchange
    const int g_stage = t + 3 < p.n_phases ? plan[t + 3].gi0 : 0, n_stage = t + 3 < p.n_phases ? plan[t + 3].len : 0;
    const uint32_t desc_word = desc_load(g_stage, n_stage);
    // (warp 1, lanes 7 and 8) the arrival counter that guards this tick's gated residual of
    // group lane - 7 of phase t - 2: the address now, the wait with the exchange
    const unsigned* bar_pp = nullptr;
    if (warp == 1 && (lane == 7 || lane == 8) && t >= 2 && (mask_pp & (1u << (lane - 7))))
      bar_pp = p.groups[plan[t - 2].gi0 + (lane - 7)].bar + 2 + parity;

    // ---- a run of dense groups (the dense baseline): nothing of the exchange machinery has
    //      work in these ticks.  Per tick: post the (empty) decision on the previous phase for
    //      the producer, stream, close with the grid barrier that keeps a dense stack in model
    //      order.  The inputs of a stack are staged before the step, so the next group's input
    //      is asked into the L2 while this group streams, and this CTA's share of it into
    //      registers while the barrier is waited for.
    auto not_gated = [&](int ph) { return ph >= p.n_phases || plan[ph].kind != 1; };
    const bool plain = dense && !mask_pp && (t == 0 || plan[t - 1].kind == 2) && not_gated(t + 1) && not_gated(t + 2);
    const unsigned mask_stream = mask_pp;   // the gated residuals this tick streams: phase t - 2
    if (plain) {
      auto x_of = [&](const PersistGroup& gg) {
        return gg.x + (long long)slot_io * gg.x_step_stride + (size_t)p.token * gg.d;
      };
      unsigned long long in[kWVecMax][4];
      WGeo q = w_geometry(&g);
      w_load_in(q, x_of(g), in);
      uint32_t dword = desc_word;   // descriptors of the phase after the next, requested at the top of the tick
      int tt = t;
      for (;;) {
        const Plan plc = plan[tt];
        const PersistGroup& gc = desc(plc.gi);
        const int gs = tt + 3 < p.n_phases ? plan[tt + 3].gi0 : 0, ns = tt + 3 < p.n_phases ? plan[tt + 3].len : 0;
        if (tt != t) dword = desc_load(gs, ns);
        if (plc.zeroer && tid < 2) gc.bar[2 * tid + (parity ^ 1u)] = 0u;
        if (tid == 0 && tt >= 1) misc->decision[(tt - 1) & 3] = (unsigned)tt << 8;
        const bool more = tt + 1 < n_ticks && plan[tt + 1].kind == 2 && not_gated(tt + 2) && not_gated(tt + 3);
        if (warp == kStatWarp && tt + 1 < n_ticks) {
          const Plan& pn = plan[tt + 1];
          if (pn.kind == 2) {
            const char* xn = reinterpret_cast<const char*>(x_of(desc(pn.gi)));
            for (int i = lane * 128; i < desc(pn.gi).d * 4; i += 32 * 128)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(xn + i));
          }
        }
        tr.mark(0);
        n = w_run(&gc, q, in, gc.y + (size_t)p.token * gc.O, true, smem, n, p.status, p.trace != nullptr);
        if (tr.acc) tr.t = clock64();
        desc_store(gs, ns, dword);   // (their latency ran under the stream)
        if (tid == 0) red_relaxed_u32(gc.bar + parity, 1u);
        if (more) {   // in flight while the barrier is waited for
          const PersistGroup& gn = desc(plan[tt + 1].gi);
          q = w_geometry(&gn);
          w_load_in(q, x_of(gn), in);
        }
        if (tid == 0) {
          grid_wait(gc.bar + parity, (unsigned)G, p, misc);
          if (cta == 0) p.gate_log[((size_t)slot_io * p.log_step_stride + plc.gi) * p.n_tokens + p.token] = 1;
          misc->stop[1] = *abort;
        }
        csync();
        tr.mark(6);
        if (misc->stop[1]) {   // decided before the barrier: the same for every warp
      async_drain();
      return;
    }
        if (!more) break;
        ++tt;
      }
      t = tt;   // the loop's increment moves on to the tick after the run
      mask_pp = 0;
      continue;
    } else {
    // ---- A. the bulk reduction of the previous tick has read its source
    if (lane == 0 || tid == kNC - 1) bulk_reduce_wait_read();   // the lanes that issue bulk reductions
    if (tid == 0) misc->fire[tp] = misc->fire[tp + 1] = 0;
    if (t >= 0 && pl.zeroer) {  // this CTA clears the group's counters for the next launch
      if (gsi) {
#pragma unroll 1
        for (int j = tid; j < k + 4; j += kNC) g.acc[(size_t)(parity ^ 1u) * (k + 4) + j] = 0ull;
      }
      if (tid < 2) g.bar[2 * tid + (parity ^ 1u)] = 0u;
    }
    if (tid == 0) misc->stop[0] = *abort;
    csync();
    if (misc->stop[0]) {   // decided before the barrier: the same for every warp
      async_drain();
      return;
    }
    tr.mark(0);
    // the statistics warp works two ticks ahead: the rows of x of phase t + 2 are requested now,
    // their statistics are published during this tick, and the other CTAs' words are collected
    // during the row passes (the inputs of a stack are staged before the step)
    if (warp == kStatWarp && t + 2 < n_ticks) stat_warp_step(smem, t + 2, true, slot_io, p.token, tag);

    // ---- B / D. (warps 5..13) pass 1 and the send of phase t + 1, beside the wait for the
    //      exchange of phase t.  Pass 1 on the tensor cores: D[term of x][column j] +=
    //      X[term][row i] P[i][j]; the rows of x are the A operand (three terms in rows 0..2), a
    //      tile of P, each of its four 8 x 8 blocks transposed by the load, is the B operand of
    //      two instructions.  Then every warp converts its own columns to fixed point and sends
    //      them off with a bulk reduction of its own into the group's accumulators.
    // chunk sequence of the tick: the basis slab of phase t + 1 for its pass 1 (given back
    // by the pass-1 warps as soon as its tiles are in registers), the basis slab of phase t once more for its
    // residual rows (the second read comes from the L2: the ring is a FIFO, and a slab kept
    // across the tick boundary would pin everything placed after it), the image slab of phase t
    const unsigned n_pf = n;
    if (gsi_f) n += pf.pchunks;
    const unsigned n_pr = n;
    if (gsi) n += pchunks;
    if (gsi_f && warp >= kP1First && warp < kStatWarp) {
      const PersistGroup& gf = desc(pf.gi);
      const int kf = kK ? kK : gf.k, KTf = kf >> 4, gclf = pf.gc_log2, wp1 = warp - kP1First;
      // partial c of this warp's tile columns kt = wp1 * tpw + s: lanes 0..3 hold, after the
      // folds below, columns 16 kt + 8 m + 2 lane + v in cacc[s][m][v]
      constexpr int kTpwMax = kK ? (kK / 16 + kP1 - 1) / kP1 : 4;
      const int tpw = kK ? kTpwMax : (KTf + kP1 - 1) / kP1;
      float cacc[kTpwMax][2][4];
      // the warps that own tile columns wait for the slab and, between them, give it back
      const int nf = min(kP1, (KTf + tpw - 1) / tpw);
      const bool p1_active = wp1 < nf && pf.pg > 0;
      bool okf = !p1_active || chunks_landed(smem, n_pf, pf.pchunks, abort);
#pragma unroll
      for (int s3 = 0; s3 < kTpwMax; ++s3)
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
          for (int v = 0; v < 4; ++v) cacc[s3][m][v] = 0.f;
      const unsigned short* xt = s_xt + ((t + 1) & 1) * 2048;
      if (okf) {
#pragma unroll 1
        for (int R = 0; R < pf.pg; ++R) {
          const uint2 ax = *reinterpret_cast<const uint2*>(xt + (R * 32 + lane) * 4);
          const uint4 a = make_uint4(ax.x, 0u, ax.y, 0u);
          const int ci = R >> gclf, rr = R - (ci << gclf);
          const unsigned char* trow = ring + s_off[(n_pf + ci) % kNB] + (size_t)rr * KTf * 512 + lane * 16;
#pragma unroll
          for (int s3 = 0; s3 < kTpwMax; ++s3) {
            const int kt = wp1 * tpw + s3;
            if (s3 < tpw && kt < KTf) {
              const uint4 w = ldsm_tile_trans(trow + kt * 512);
              mma_bf16(cacc[s3][0], a, w.x, w.y);
              mma_bf16(cacc[s3][1], a, w.z, w.w);
            }
          }
        }
      }
      if (okf && p1_active && lane == 0) {   // (every tile of the slab is in registers: the last mma has issued)
        const uint32_t share = unit_share(wp1, nf);
#pragma unroll 1
        for (int c = 0; c < pf.pchunks; ++c) mbar_arrive_n(&empty[(n_pf + c) % kNB], share);
      }
      // the three terms of x sit in rows 0..2 = lanes 0-3, 4-7, 8-11: fold them onto lanes 0-3
#pragma unroll
      for (int s3 = 0; s3 < kTpwMax; ++s3)
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            float z = cacc[s3][m][v];
            z += __shfl_down_sync(0xffffffffu, z, 4) + __shfl_down_sync(0xffffffffu, z, 8);
            cacc[s3][m][v] = z;
          }
      if (!okf && !*abort) fail(p, misc, 5);
      // fixed-point scale: |partial c_j| <= amax * rows * max|P| < 2^e
      const unsigned amax_f = misc->amax_bits[(t + 1) & 1];
      const float bound = __uint_as_float(amax_f) * (float)gf.p_rows * gf.pmax;
      double scale = 0.0;
      if (amax_f < 0x7f800000u && bound > 0.f && bound < 3.0e38f)
        scale = pow2d(43 - (max((int)((__float_as_uint(bound) >> 23) & 0xFFu), 1) - 126));
      if (pf.pg > 0 && wp1 * tpw < KTf) {
        unsigned long long* acc_f = gf.acc + (size_t)parity * (kf + 4);
        if (lane < 4) {
#pragma unroll
          for (int s3 = 0; s3 < kTpwMax; ++s3) {
            const int kt = wp1 * tpw + s3;
            if (s3 < tpw && kt < KTf) {
#pragma unroll
              for (int m = 0; m < 2; ++m)
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                  const long long fx = scale != 0.0 ? __double2ll_rn((double)cacc[s3][m][v] * scale) : 0ll;
                  s_fx[16 * kt + 8 * m + 2 * lane + v] = kOne + (unsigned long long)fx;
                }
            }
          }
        }
        __syncwarp();
        if (lane == 0) {
          const int c0 = 16 * wp1 * tpw, c1 = min(kf, c0 + 16 * tpw);
          bulk_reduce_add_u64(acc_f + c0, s_fx + c0, (uint32_t)(c1 - c0) * 8);
        }
      }
    }
    if (gsi_f && tid == kNC - 1 && pf.pg > 0) {   // ||x||^2 of phase t + 1 over this CTA's rows
      const PersistGroup& gf = desc(pf.gi);
      const int kf = kK ? kK : gf.k;
      const unsigned amax_f = misc->amax_bits[(t + 1) & 1];
      const double amax = (double)__uint_as_float(amax_f);
      const float bound = __uint_as_float(amax_f) * (float)gf.p_rows * gf.pmax;
      const bool fin = amax_f < 0x7f800000u && bound > 0.f && bound < 3.0e38f;
      const double scale_x2 = fin ? pow2d(43 - exp_above(amax * amax * (double)gf.p_rows)) : 0.0;
      const long long v = scale_x2 != 0.0 ? __double2ll_rn((double)misc->x2_part[(t + 1) & 1] * scale_x2) : 0ll;
      s_fx[kf] = kOne + (unsigned long long)v;
      s_fx[kf + 1] = 0ull;
      bulk_reduce_add_u64(gf.acc + (size_t)parity * (kf + 4) + kf, s_fx + kf, 16u);
    }
    if (warp == kStatWarp && t + 2 < n_ticks) stat_warp_step(smem, t + 2, false, slot_io, p.token, tag);
    tr.mark(3);

    // the scale of the sums of phase t (sent a tick ago), and whether its token is finite
    bool nonfinite = false;
    double inv_scale = 0.0;
    if (gsi) {
      const unsigned amax_bits = misc->amax_bits[t & 1];
      nonfinite = amax_bits >= 0x7f800000u;
      const float bound = __uint_as_float(amax_bits) * (float)g.p_rows * g.pmax;
      if (!nonfinite && bound > 0.f && bound < 3.0e38f)
        inv_scale = pow2d(max((int)((__float_as_uint(bound) >> 23) & 0xFFu), 1) - 126 - 43);
    }

    // ---- E. wait until every contributing CTA has been added: four warps poll a quarter of
    //      the accumulators of c each (contiguous words, all loads of a lane in flight together,
    //      one round trip per attempt) and leave c as three bf16 terms in operand order;
    //      warp 1 polls the scalars: lane 0 this phase's ||x||^2, lanes 1+2u / 2+2u the
    //      previous phase's ||r||^2 and published ||x||^2 of its group u.
    if (gsi && (warp == 0 || (warp >= 2 && warp <= 4))) {
      constexpr int kWpl = kK ? (kK + 127) / 128 : 4;   // words per lane
      const int q4 = warp == 0 ? 0 : warp - 1;          // this warp's quarter of the words
      unsigned long long w[kWpl];
      unsigned it = 0;
      bool done = false;
      while (!done) {
        bool all = true;
#pragma unroll
        for (int i = 0; i < kWpl; ++i) {
          const int j = (q4 + 4 * i) * 32 + lane;
          w[i] = j < k ? ld_relaxed_u64(acc + j) : ((unsigned long long)n_contrib << kCountShift);
        }
#pragma unroll
        for (int i = 0; i < kWpl; ++i)
          all = all && ((unsigned)((w[i] + (kOne >> 1)) >> kCountShift) == (unsigned)n_contrib);
        done = __all_sync(0xffffffffu, all);
        if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
          if (!*abort && lane == 0) fail(p, misc, 6);
          break;
        }
      }
#pragma unroll
      for (int i = 0; i < kWpl; ++i) {
        const int j = (q4 + 4 * i) * 32 + lane;
        if (j < k) {
          const long long val = (long long)(w[i] - ((unsigned long long)n_contrib << kCountShift));
          unsigned short tm[3];
          split3((float)((double)val * inv_scale), tm);
          const int slot = term_slot(j >> 4, j & 15, 0);
          s_cb[slot] = tm[0];
          s_cb[slot + 16] = tm[1];   // the next term is the next column of the operand: four lanes on
          s_cb[slot + 32] = tm[2];
        }
      }
    }
    if (warp == 1) {
      // lane 0: this phase's ||x||^2 (an accumulator: arrivals in the upper bits); lanes
      // 1 + 2u / 2 + 2u: the previous phase's ||r||^2 (accumulator) and its gate threshold
      // (tagged word) of group u
      // (on CTA 0, which writes the logs, lanes 5 + u also fetch the group's published ||x||^2)
      const int u = lane <= 4 ? (lane - 1) >> 1 : lane - 5;
      const bool live_u = u >= 0 && u < len_p && !(desc(g_p + u).flags & GSI_FLAG_DENSE);
      const bool settle = lane >= 1 && lane <= 4 && live_u;
      const PersistGroup& gs = desc(g_p + (u & 1));   // read only when `live_u`
      const bool w_x2 = gsi && lane == 0, w_r2 = settle && (lane & 1);
      const bool w_thr = (settle && !(lane & 1)) || (cta == 0 && lane >= 5 && lane <= 6 && live_u);
      // lanes 7, 8: the arrivals before the gated residual this tick streams (phase t - 2, group
      // lane - 7): every CTA has made its r and image rows visible (they arrived a tick ago)
      const bool w_bar = bar_pp != nullptr;
      const unsigned long long* wp = w_x2   ? acc + k
                                     : w_r2 ? gs.acc + (size_t)parity * (gs.k + 4) + gs.k + 2
                                            : gs.pub + (lane <= 4 ? 1 : 0);
      const unsigned want = w_x2 ? (unsigned)n_contrib : (unsigned)gs.n_contrib;
      unsigned long long w = 0;
      unsigned it = 0;
      bool done = false;
      while (!done) {
        bool mine = true;
        if (w_x2 || w_r2 || w_thr) {
          w = ld_relaxed_u64(wp);
          mine = w_thr ? (unsigned)(w >> 63) == tag
                       : (unsigned)((w + (kOne >> 1)) >> kCountShift) == want;
        } else if (w_bar) {
          mine = ld_relaxed_u32(bar_pp) >= (unsigned)G;
        }
        done = __all_sync(0xffffffffu, mine);
        if (!done && (++it > p.spin_limit || ((it & 1023u) == 0 && *abort))) {
          if (!*abort && lane == 0) fail(p, misc, 7);
          break;
        }
      }
      if (w_bar) __threadfence();   // acquire: the barrier below hands the visibility on to the CTA
      if (w_x2) {
        const long long val = (long long)(w - ((unsigned long long)n_contrib << kCountShift));
        const double amax = (double)__uint_as_float(misc->amax_bits[t & 1]);
        const double x2 = nonfinite ? __longlong_as_double(0x7ff8000000000000ll)
                          : val > 0 ? (double)val * pow2d(exp_above(amax * amax * (double)g.p_rows) - 43)
                                    : 0.0;
        misc->x2 = x2;
        if (lc == 0) {
          // Every CTA settles this group's gate in the next tick by comparing integers:
          // ||r||^2 < eps^2 ||x||^2 (both sides >= 0; false for x = 0) in the fixed-point
          // units 2^(e - 44) of ||r||^2 is sum < ceil(eps^2 ||x||^2 2^(44 - e)).  Bit 62 marks a
          // non-finite token (never fast, never streamed).  ||x||^2 itself goes out for rho.
          const double eps = (double)g.eps;
          const double thr = fmin(ceil(eps * eps * x2 * pow2d(44 - (x2 > 0.0 ? exp_above(x2) : 0))), 2305843009213693952.0);
          const unsigned long long tw = nonfinite ? (1ull << 62) : (unsigned long long)thr;
          st_relaxed_u64(g.pub + 1, tw | ((unsigned long long)tag << 63));
          st_relaxed_u64(g.pub, ((unsigned long long)__double_as_longlong(x2) & ~(1ull << 63)) |
                                    ((unsigned long long)tag << 63));
        }
      }
      // the lane that holds ||r||^2 of group u takes the threshold from its neighbour
      const unsigned long long w_nb = __shfl_down_sync(0xffffffffu, w, 1);
      const unsigned long long wx = __shfl_sync(0xffffffffu, w, 5 + (u & 1));
      if (w_r2) {
        const unsigned long long val = w - ((unsigned long long)want << kCountShift);
        const bool finite = !(w_nb & (1ull << 62));
        const bool fast = finite && val < (w_nb & ((1ull << 62) - 1));
        misc->fire[tp + u] = (!fast && finite && !(gs.flags & GSI_FLAG_STATIC_PROJECTION)) ? 1 : 0;
        if (cta == 0) {   // the logs: rho from ||r||^2 2^-e and ||x||^2 2^-e, both in the float range
          const double x2 = __longlong_as_double((long long)(wx & ~(1ull << 63)));
          const int ex = x2 > 0.0 ? exp_above(x2) : 0;
          const size_t at = ((size_t)slot_io * p.log_step_stride + (g_p + u)) * p.n_tokens + p.token;
          p.gate_log[at] = fast ? 0 : 1;
          if (p.rho_log)
            p.rho_log[at] = finite ? sqrtf(__fdividef((float)((double)val * 5.6843418860808015e-14),
                                                      (float)(x2 * pow2d(-ex))))
                                   : __int_as_float(0x7fc00000);
        }
      }
    }
    desc_store(g_stage, n_stage, desc_word);
    if (tid == 0) misc->stop[1] = *abort;
    csync();
    tr.mark(4);
    if (misc->stop[1]) {   // decided before the barrier: the same for every warp
      async_drain();
      return;
    }

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
    // (this warp then fetches the words of the other CTAs for the next phase: the loads fly
    // during its row units, the check comes after them)
    unsigned xw[kXmaxWords];
    const bool xmax_next = warp == kStatWarp && t + 2 < n_ticks && plan[t + 2].kind == 1;
    if (xmax_next) xmax_issue(desc(plan[t + 2].gi).xmax, plan[t + 2].n_contrib, xw);

    // ---- G / I. the row passes on the tensor cores, one copy of the code for both: part 0 the
    //      residual rows of the basis slab (still in the ring), part 1 the image rows.  A unit
    //      is a tile row (16 matrix rows): D[row][term of c] += T[row][column] C[column][term],
    //      the tiles as they lie in the ring are the A operand, c (three terms in columns
    //      0..2) the B operand.  Units are dealt round-robin over the joint numbering of both
    //      parts, so the warps are loaded evenly.
#pragma unroll 1
    for (int part = 0; part < 2; ++part) {
      if (!gsi) continue;
      const bool image = part == 1;
      const int ngroups = image ? og : pg;
      const int id0 = image ? pg : 0;
      const unsigned n0 = image ? n : n_pr;
      const int row_base = image ? pl.o0 : pl.p0, row_end = image ? g.O : g.d;
      float* out = image ? g.y + (size_t)p.token * g.O : g.r;
      const bool f8 = image && (g.flags & GSI_FLAG_FP8_IMAGE);
      if (image) n += ochunks;
      float sr = 0.f;
      // A warp touches only the chunks its units lie in: it waits for the chunk, runs the unit
      // and hands in the unit's share of the chunk's arrivals (the chunk goes back to the
      // producer when all its units are done).  The image slab need not be resident as a whole:
      // its chunks stream through the space that the basis slab of the next phase leaves.
      if (ok) {
        int id = warp;
        if (id < id0) id += ((id0 - id + kNW - 1) / kNW) * kNW;
#pragma unroll 1
        for (; id < id0 + ngroups && ok; id += kNW) {
          const int R = id - id0;
          const int ci = R >> gcl, rr = R - (ci << gcl);
          const unsigned seq = n0 + ci;
          // (the outcome is taken for the warp as a whole: lanes must not part ways here)
          if (!__all_sync(0xffffffffu, mbar_wait(&full_b[seq % kNB], (seq / kNB) & 1u, abort))) ok = false;
          if (!ok) break;
          const unsigned char* cb = reinterpret_cast<const unsigned char*>(s_cb) + lane * 8;
          float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
          float sc_lo = 1.f, sc_hi = 1.f;   // FP8 image: the scales of rows lg and lg + 8
          if (f8) {
            // tiles of one byte per element, expanded to bf16 in registers; the row scales follow the tiles
            const unsigned char* trow8 = ring + s_off[(n0 + ci) % kNB] + (size_t)rr * (KT * 256 + 64);
            sc_lo = *reinterpret_cast<const float*>(trow8 + KT * 256 + lg * 4);
            sc_hi = *reinterpret_cast<const float*>(trow8 + KT * 256 + lg * 4 + 32);
            trow8 += lane * 8;
#pragma unroll 2
            for (int K = 0; K < KT; K += 2) {
              const uint2 q0 = *reinterpret_cast<const uint2*>(trow8 + K * 256);
              const uint2 b0 = *reinterpret_cast<const uint2*>(cb + K * 256);
              const uint2 q1 = *reinterpret_cast<const uint2*>(trow8 + K * 256 + 256);
              const uint2 b1 = *reinterpret_cast<const uint2*>(cb + K * 256 + 256);
              const uint4 a0 = make_uint4(e4m3x2_to_bf16x2(q0.x), e4m3x2_to_bf16x2(q0.x >> 16),
                                          e4m3x2_to_bf16x2(q0.y), e4m3x2_to_bf16x2(q0.y >> 16));
              const uint4 a1 = make_uint4(e4m3x2_to_bf16x2(q1.x), e4m3x2_to_bf16x2(q1.x >> 16),
                                          e4m3x2_to_bf16x2(q1.y), e4m3x2_to_bf16x2(q1.y >> 16));
              mma_bf16(d0, a0, b0.x, b0.y);
              mma_bf16(d1, a1, b1.x, b1.y);
            }
          } else {
            const unsigned char* trow = ring + s_off[(n0 + ci) % kNB] + (size_t)rr * KT * 512 + lane * 16;
#pragma unroll 2
            for (int K = 0; K < KT; K += 2) {   // two chains of dependent instructions
              const uint4 a0 = ldsm_tile(trow + K * 512);
              const uint2 b0 = *reinterpret_cast<const uint2*>(cb + K * 256);
              const uint4 a1 = ldsm_tile(trow + K * 512 + 512);
              const uint2 b1 = *reinterpret_cast<const uint2*>(cb + K * 256 + 256);
              mma_bf16(d0, a0, b0.x, b0.y);
              mma_bf16(d1, a1, b1.x, b1.y);
            }
          }
          // the unit's tiles are in registers (the last mma has issued): its share of the chunk goes back
          if (lane == 0) mbar_arrive_n(&empty[seq % kNB], unit_share(rr, min(1 << gcl, ngroups - (ci << gcl))));
          // columns 0, 1 (lane pair 0) and 2 (lane pair 1) of D are the three terms of c
          const float lo = d0[0] + d1[0], lo1 = d0[1] + d1[1], hi = d0[2] + d1[2], hi1 = d0[3] + d1[3];
          const float lo2 = __shfl_down_sync(0xffffffffu, lo, 1), hi2 = __shfl_down_sync(0xffffffffu, hi, 1);
          if (lt == 0) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const float dot = h ? ((hi + hi1) + hi2) * sc_hi : ((lo + lo1) + lo2) * sc_lo;
              const int row = R * 16 + lg + 8 * h;
              if (row_base + row < row_end) {
                if (image) {
                  out[row_base + row] = nonfinite ? __int_as_float(0x7fc00000) : dot;
                } else {
                  const float rv = s_x[row] - dot;
                  out[row_base + row] = rv;
                  sr = fmaf(rv, rv, sr);
                }
              }
            }
          }
        }
        if (image) tr.mark(7);
      }
      if (!image) {
        // ||r||^2: every warp adds its rows' share, in the fixed-point units 2^(e - 44) of the
        // exchange, to one word of shared memory whose upper bits count the warps (integers: the
        // sum does not depend on who finished first; no fence: the one atomic carries value and
        // count); the warp that arrives last sends the CTA's share as one atomic; the next
        // tick's exchange settles the gate.  A share is at most 2^45, so the sum of all CTAs
        // stays below 2^53; a partial that large (||r||^2 > 2 ||x||^2) fires for every sensible eps
        sr = warp_sum(sr);
        if (lane == 0) {
          double vd = (double)sr * pow2d(44 - (x2_own > 0.0 ? exp_above(x2_own) : 0));
          if (!(vd < 35184372088832.0)) vd = 35184372088832.0;
          if (!(vd >= 0.0)) vd = 0.0;
          const unsigned long long mine = kOne + (unsigned long long)__double2ll_rn(vd);
          const unsigned long long before = atomicAdd(&misc->r2_acc, mine);
          if ((unsigned)((before + mine) >> kCountShift) == (unsigned)kNW) {
            misc->r2_acc = 0ull;   // (next used behind two barriers)
            if (pg > 0) {
              const unsigned long long sum = before + mine - ((unsigned long long)kNW << kCountShift);
              red_add_u64(acc + k + 2, kOne + (sum < 35184372088832ull ? sum : 35184372088832ull));
            }
          }
        }
      }
      tr.mark(image ? 8 : 5);
    }
    if (!ok && !*abort) fail(p, misc, 8);   // (the CTA leaves together, behind the next barrier)
    if (xmax_next) xmax_collect(smem, t + 2, tag, p.spin_limit, p.status, xw[0], xw[1], xw[2], xw[3], xw[4]);

    mask_pp = mask_p;
    }

    // ---- H. the W streams of the tick, one call site, after the row passes (little of the
    //      tick's state is alive here): the gated residuals of the phase before the previous
    //      one, then this phase's own stream if it is a dense group (followed by a grid barrier
    //      that keeps a dense stack in model order).
    if (mask_stream || dense) {
      const int len_pp = plan[t - 2 >= 0 ? t - 2 : 0].len, g_pp = plan[t - 2 >= 0 ? t - 2 : 0].gi0;
#pragma unroll 1
      for (int u = 0; u < 3; ++u) {
        const PersistGroup* gw = nullptr;
        if (u < 2) {
          if (u < len_pp && (mask_stream & (1u << u))) gw = p.groups + g_pp + u;
        } else if (dense) {
          gw = &desc(plan[t].gi);
        }
        if (!gw) continue;
        // (a gated group's r and image rows are visible: warp 1 waited for every CTA's arrival
        // during this tick's exchange)
        const float* src = u < 2 ? gw->r
                                 : gw->x + (long long)slot_io * gw->x_step_stride + (size_t)p.token * gw->d;
        tr.mark(9);
        n = w_stream(gw, src, gw->y + (size_t)p.token * gw->O, u == 2, smem, n, p.status, p.trace != nullptr);
        if (tr.acc) tr.t = clock64();
        if (u == 2) {
          if (tid == 0) {
            red_relaxed_u32(gw->bar + parity, 1u);
            grid_wait(gw->bar + parity, (unsigned)G, p, misc);
            if (cta == 0)
              p.gate_log[((size_t)slot_io * p.log_step_stride + plan[t].gi) * p.n_tokens + p.token] = 1;
          }
          csync();
        }
      }
      tr.mark(6);
    }
  }
  async_drain();
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
    misc->r2_acc = 0ull;
    // shared memory keeps what the previous launch on this SM left: the producer must not
    // mistake an old decision for this launch's
    misc->fire[0] = misc->fire[1] = misc->fire[2] = misc->fire[3] = 0;
    misc->decision[0] = misc->decision[1] = misc->decision[2] = misc->decision[3] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  make_plan<kPairs, kK>(p, smem);
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
