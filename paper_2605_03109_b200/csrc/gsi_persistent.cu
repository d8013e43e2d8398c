// Persistent decode-step kernel: every group of the stack in ONE launch.
//
// One CTA per SM.  Each CTA owns a fixed slab of rows of every basis P and of
// every (concatenated) image W_P.  A producer warp streams those slabs from HBM
// into a ring of shared-memory slots with bulk async copies, in program order
// and independent of the data-dependent steps (weight addresses never depend
// on x), so the next group's weights arrive while the current group waits on
// its cross-CTA exchanges.  Twelve consumer warps run Algorithm 1 per group:
//
//   pass 1     partial c = P_slab^T x_slab                     (line 1)
//   exchange 1 c = sum over CTAs, by 64-bit fixed-point atomics whose words
//              also count arrivals (no separate flag, no fence, order-free and
//              therefore bit-reproducible)
//   pass 2     r_slab = x_slab - P_slab c, partial ||r||^2      (lines 2-3)
//   image      y_rows = W_P,rows c                              (line 5)
//   exchange 2 every CTA publishes (step tag | partial ||r||^2) in one 64-bit
//              word with release semantics; every CTA sums the words in a fixed
//              order and takes the same gate decision           (line 4)
//   gated      y_rows += W_rows r, W streamed with 256-bit loads, then a grid
//              barrier                                          (Eq. (3.2))
//
// Every wait is bounded; a wait that gives up records GSI_ERR_TIMEOUT in the
// status word, the CTA drains its copies in flight and returns.
#include <cooperative_groups.h>

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
constexpr unsigned kSpinLimit = 1u << 22;
constexpr int kCountShift = 54;

// shared memory map (bytes)
constexpr int kOffBar = 0;          // full[kSlots], empty[kSlots]
constexpr int kOffMisc = 256;       // abort flag, scalars
constexpr int kOffX = 512;          // x of this CTA's basis rows      (kPersistMaxPRows floats)
constexpr int kOffC = 1024;         // c                                (512 floats)
constexpr int kOffVals = 3072;      // exchange-2 values                (256 floats)
constexpr int kOffRed = 4096;       // cross-warp scratch               (kNW*512 floats)
constexpr int kOffRq = kOffRed + kNW * 512 * 4;   // staged r, 4 interleaved quarters (16 KB)
constexpr int kOffYacc = kOffRq + 16384;          // per-row accumulators (kPersistMaxORows floats)
constexpr int kOffRing = ((kOffYacc + kPersistMaxORows * 4 + 1023) / 1024) * 1024;
constexpr int kSmemBytes = kOffRing + kSlots * kChunk;
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 CTA");

struct Misc {
  int abort;
  int gate;
  float amax;
  float sum2;
  int nonfinite;
  float sr;
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
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_u32(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
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

// Rows [r0, r1) of a slab, in chunks of `rc` rows; returns the chunk count.
__device__ __forceinline__ int n_chunks(int rows, int rc) { return (rows + rc - 1) / rc; }

struct Slab {
  int p0, p1;  // basis rows owned by this CTA
  int o0, o1;  // rows of the concatenated maps owned by this CTA
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
    const Slab s = slab_of(g, blockIdx.x);
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
  unsigned parity, tag;
  unsigned n;  // ring sequence number, advances exactly as in producer()
};

// One group.  Returns false when the CTA must stop (a wait gave up).
template <int VPL>
__device__ bool group_phase(const PersistParams& p, unsigned char* smem, Misc* misc, Ctx& ctx,
                            int gi) {
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty = full + kSlots;
  float* s_x = reinterpret_cast<float*>(smem + kOffX);
  float* s_c = reinterpret_cast<float*>(smem + kOffC);
  float* s_vals = reinterpret_cast<float*>(smem + kOffVals);
  float* s_red = reinterpret_cast<float*>(smem + kOffRed);
  float4* s_rq = reinterpret_cast<float4*>(smem + kOffRq);
  float* s_yacc = reinterpret_cast<float*>(smem + kOffYacc);
  unsigned char* ring = smem + kOffRing;
  volatile int* abort = &misc->abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int slot_io = ctx.slot_io;
  const unsigned parity = ctx.parity, tag = ctx.tag;
  unsigned& n = ctx.n;
  {
    const PersistGroup& g = p.groups[gi];
    const int KV = g.k / 8;
    const Slab s = slab_of(g, cta);
    const float* x = g.x + (long long)slot_io * g.x_step_stride;
    const bool dense = g.flags & GSI_FLAG_DENSE;
    int gate = 1;
    const float* rsrc = x;

    // make the next group's activations L2-resident while this one runs
    if (gi + 1 < p.n_groups) {
      const PersistGroup& gn = p.groups[gi + 1];
      const char* xn = reinterpret_cast<const char*>(gn.x + (long long)slot_io * gn.x_step_stride);
      const int lines = (gn.d * 4 + 127) / 128;
      for (int l = cta * kNC + tid; l < lines; l += G * kNC) prefetch_l2(xn + (size_t)l * 128);
    }

    if (!dense) {
      const int k = g.k;
      const int LPR = KV < 32 ? KV : 32, RPP = 32 / LPR;
      const int sub = lane / LPR, cl = lane % LPR;
      const int rc = kChunk / (k * 2);
      const int n_contrib = (g.d + g.p_rows - 1) / g.p_rows;
      unsigned long long* acc = g.acc_c + (size_t)parity * k;

      // ---- A. statistics of x (every CTA, the whole vector): max |x|, sum x^2
      float amax = 0.f, sum2 = 0.f;
      int bad = 0;
      for (int i4 = tid; i4 < g.d / 4; i4 += kNC) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(x) + i4);
        const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          amax = fmaxf(amax, fabsf(e[q]));
          sum2 = fmaf(e[q], e[q], sum2);
          bad |= !(fabsf(e[q]) <= 3.0e38f);
          const int i = i4 * 4 + q;
          if (i >= s.p0 && i < s.p1) s_x[i - s.p0] = e[q];
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        sum2 += __shfl_xor_sync(0xffffffffu, sum2, o);
        bad |= __shfl_xor_sync(0xffffffffu, bad, o);
      }
      if (lane == 0) {
        s_red[warp * 4 + 0] = amax;
        s_red[warp * 4 + 1] = sum2;
        s_red[warp * 4 + 2] = (float)bad;
      }
      if (cta == gi % G) {  // clear the accumulators the NEXT step will use
        for (int j = tid; j < k; j += kNC) g.acc_c[(size_t)(parity ^ 1u) * k + j] = 0ull;
        if (tid == 0) g.bar[parity ^ 1u] = 0u;
      }
      csync();
      if (tid == 0) {
        float a = 0.f, q = 0.f, b = 0.f;
        for (int w = 0; w < kNW; ++w) {
          a = fmaxf(a, s_red[w * 4]);
          q += s_red[w * 4 + 1];
          b += s_red[w * 4 + 2];
        }
        misc->amax = a;
        misc->sum2 = q;
        misc->nonfinite = b != 0.f;
      }
      csync();
      const int nonfinite = misc->nonfinite;
      // fixed-point scale: |partial c_j| <= amax * rows * max|P| < 2^e
      double scale = 0.0, inv_scale = 0.0;
      {
        const float bound = misc->amax * (float)g.p_rows * __ldg(g.pmax);
        if (!nonfinite && bound > 0.f && bound < 3.0e38f) {
          int e;
          frexpf(bound, &e);
          scale = ldexp(1.0, 43 - e);
          inv_scale = ldexp(1.0, e - 43);
        }
      }

      // ---- B. pass 1: partial c over this CTA's basis rows
      const unsigned n_p0 = n;
      const int pchunks = n_chunks(s.p1 - s.p0, rc);
      float accv[VPL][8];
#pragma unroll
      for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 8; ++e) accv[v][e] = 0.f;
      bool ok = true;
      for (int ci = 0; ci < pchunks; ++ci) {
        const unsigned sl = (n_p0 + ci) % kSlots, ph = ((n_p0 + ci) / kSlots) & 1u;
        ok = ok && mbar_wait(&full[sl], ph, abort);
        if (!ok) break;
        const uint4* tile = reinterpret_cast<const uint4*>(ring + (size_t)sl * kChunk);
        const int r_lo = ci * rc, rows = min(rc, s.p1 - s.p0 - r_lo);
        for (int base = warp * RPP; base < rows; base += kNW * RPP) {
          const int row = base + sub;
          if (row < rows) {
            const float xv = s_x[r_lo + row];
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
              float p8[8];
              unpack_bf16x8(tile[(size_t)row * KV + cl + v * LPR], p8);
#pragma unroll
              for (int e = 0; e < 8; ++e) accv[v][e] = fmaf(p8[e], xv, accv[v][e]);
            }
          }
        }
      }
      if (!ok && !*abort) fail(p, misc);
      for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int v = 0; v < VPL; ++v)
#pragma unroll
          for (int e = 0; e < 8; ++e) accv[v][e] += __shfl_xor_sync(0xffffffffu, accv[v][e], o);
      }
      if (sub == 0) {
#pragma unroll
        for (int v = 0; v < VPL; ++v)
#pragma unroll
          for (int e = 0; e < 8; ++e) s_red[warp * 512 + (cl + v * LPR) * 8 + e] = accv[v][e];
      }
      csync();
      if (*abort) return false;
      if (s.p1 > s.p0) {
        for (int j = tid; j < k; j += kNC) {
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < kNW; ++w) sum += s_red[w * 512 + j];
          const long long q = scale != 0.0 ? __double2ll_rn((double)sum * scale) : 0ll;
          red_add_u64(acc + j, (1ull << kCountShift) + (unsigned long long)q);
        }
      }

      // ---- C. exchange 1: wait until every contributing CTA has been added
      for (int j = tid; j < k; j += kNC) {
        unsigned long long w = 0;
        unsigned it = 0;
        for (;;) {
          w = ld_relaxed_u64(acc + j);
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

      // ---- D. pass 2 (residual rows) and the image rows
      float c8[VPL][8];
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const float4 a = *reinterpret_cast<const float4*>(s_c + (cl + v * LPR) * 8);
        const float4 b = *reinterpret_cast<const float4*>(s_c + (cl + v * LPR) * 8 + 4);
        c8[v][0] = a.x; c8[v][1] = a.y; c8[v][2] = a.z; c8[v][3] = a.w;
        c8[v][4] = b.x; c8[v][5] = b.y; c8[v][6] = b.z; c8[v][7] = b.w;
      }
      float sr = 0.f;
      for (int ci = 0; ci < pchunks; ++ci) {
        const unsigned sl = (n_p0 + ci) % kSlots;
        const uint4* tile = reinterpret_cast<const uint4*>(ring + (size_t)sl * kChunk);
        const int r_lo = ci * rc, rows = min(rc, s.p1 - s.p0 - r_lo);
        for (int base = warp * RPP; base < rows; base += kNW * RPP) {
          const int row = base + sub;
          float dot = 0.f;
          if (row < rows) {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
              float p8[8];
              unpack_bf16x8(tile[(size_t)row * KV + cl + v * LPR], p8);
#pragma unroll
              for (int e = 0; e < 8; ++e) dot = fmaf(p8[e], c8[v][e], dot);
            }
          }
          for (int o = LPR >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          if (row < rows && cl == 0) {
            const float rv = s_x[r_lo + row] - dot;
            g.r[s.p0 + r_lo + row] = rv;
            sr = fmaf(rv, rv, sr);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[sl]);
      }
      n += pchunks;
      const int ochunks = n_chunks(s.o1 - s.o0, rc);
      for (int ci = 0; ci < ochunks; ++ci) {
        const unsigned sl = (n + ci) % kSlots, ph = ((n + ci) / kSlots) & 1u;
        ok = ok && mbar_wait(&full[sl], ph, abort);
        if (!ok) break;
        const uint4* tile = reinterpret_cast<const uint4*>(ring + (size_t)sl * kChunk);
        const int r_lo = ci * rc, rows = min(rc, s.o1 - s.o0 - r_lo);
        for (int base = warp * RPP; base < rows; base += kNW * RPP) {
          const int row = base + sub;
          float dot = 0.f;
          if (row < rows) {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
              float p8[8];
              unpack_bf16x8(tile[(size_t)row * KV + cl + v * LPR], p8);
#pragma unroll
              for (int e = 0; e < 8; ++e) dot = fmaf(p8[e], c8[v][e], dot);
            }
          }
          for (int o = LPR >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          if (row < rows && cl == 0)
            g.y[s.o0 + r_lo + row] = nonfinite ? __int_as_float(0x7fc00000) : dot;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[sl]);
      }
      if (!ok && !*abort) fail(p, misc);
      n += ochunks;
      sr = warp_sum(sr);
      if (lane == 0) s_red[warp] = sr;
      csync();
      if (*abort) return false;

      // ---- E. exchange 2: publish, collect, decide
      if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < kNW; ++w) t += s_red[w];
        // release: this CTA's y and r rows are visible to whoever reads the word
        st_release_u64(g.slot_r + cta,
                       ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(t));
      }
      for (int t = tid; t < G; t += kNC) {
        unsigned long long w = 0;
        unsigned it = 0;
        for (;;) {
          w = ld_relaxed_u64(g.slot_r + t);
          if ((unsigned)(w >> 32) == tag) break;
          if (++it > kSpinLimit || ((it & 1023u) == 0 && *abort)) {
            if (!*abort) fail(p, misc);
            break;
          }
        }
        s_vals[t] = __uint_as_float((unsigned)w);
      }
      __threadfence();  // acquire side of the published words
      csync();
      if (*abort) return false;
      if (tid == 0) {
        double srt = 0.0;
        for (int t = 0; t < G; ++t) srt += (double)s_vals[t];
        const double nr = sqrt(srt), nx = sqrt((double)misc->sum2);
        const bool fast = !nonfinite && (nr < (double)g.eps * nx);
        misc->gate = fast ? 0 : 1;
        if (cta == 0) {
          const size_t at = (size_t)slot_io * p.log_step_stride + gi;
          p.gate_log[at] = fast ? 0 : 1;
          if (p.rho_log) p.rho_log[at] = nonfinite ? __int_as_float(0x7fc00000) : (float)(nr / nx);
        }
      }
      csync();
      gate = misc->gate && !(g.flags & GSI_FLAG_STATIC_PROJECTION) && !nonfinite;
      rsrc = g.r;
    } else {
      if (cta == gi % G && tid == 0) g.bar[parity ^ 1u] = 0u;
      if (cta == 0 && tid == 0) p.gate_log[(size_t)slot_io * p.log_step_stride + gi] = 1;
    }

    // ---- F. gated residual: y_rows (+)= W_rows . r   (dense baseline: r := x)
    if (gate) {
      const int rows = s.o1 - s.o0;
      const int nsl = (g.d + kSlice - 1) / kSlice;
      for (int sl = 0; sl < nsl; ++sl) {
        const int c0 = sl * kSlice, cols = min(kSlice, g.d - c0), nv = cols / 16;
        csync();
        for (int v = tid; v < nv; v += kNC) {
          const float4* src = reinterpret_cast<const float4*>(rsrc + c0 + v * 16);
#pragma unroll
          for (int q = 0; q < 4; ++q) s_rq[q * 256 + v] = __ldcg(src + q);
        }
        csync();
        for (int rw = warp; rw < rows; rw += kNW) {
          const int a = s.o0 + rw;
          int j = 0;
          while (j + 1 < g.n_maps && a >= g.off[j + 1]) ++j;
          const uint16_t* wrow = g.W[j] + (size_t)(a - g.off[j]) * g.d + c0;
          float acc = 0.f;
          for (int v0 = lane; v0 < nv; v0 += 4 * 32) {
            uint32_t w[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int v = v0 + u * 32;
              if (v < nv) ld256_stream(wrow + (size_t)v * 16, w[u]);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int v = v0 + u * 32;
              if (v < nv) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const float4 rr = s_rq[q * 256 + v];
                  const uint32_t lo = w[u][2 * q], hi = w[u][2 * q + 1];
                  acc = fmaf(__uint_as_float(lo << 16), rr.x, acc);
                  acc = fmaf(__uint_as_float(lo & 0xFFFF0000u), rr.y, acc);
                  acc = fmaf(__uint_as_float(hi << 16), rr.z, acc);
                  acc = fmaf(__uint_as_float(hi & 0xFFFF0000u), rr.w, acc);
                }
              }
            }
          }
          acc = warp_sum(acc);
          if (lane == 0) s_yacc[rw] = (sl == 0 ? 0.f : s_yacc[rw]) + acc;
        }
      }
      __syncwarp();
      for (int rw = warp; rw < rows; rw += kNW) {
        if (lane == 0) {
          float* yp = g.y + s.o0 + rw;
          *yp = dense ? s_yacc[rw] : (*yp + s_yacc[rw]);
        }
      }
      // grid barrier: the next group may read every row of y
      csync();
      if (tid == 0) {
        red_release_u32(g.bar + parity, 1u);
        unsigned it = 0;
        while (ld_acquire_u32(g.bar + parity) < (unsigned)G) {
          if (++it > kSpinLimit || *abort) {
            if (!*abort) fail(p, misc);
            break;
          }
        }
      }
      csync();
      if (*abort) return false;
    }
  }
  return true;
}

__device__ void consumer(const PersistParams& p, unsigned char* smem, Misc* misc) {
  Ctx ctx;
  ctx.step = p.use_counter ? *p.step : 0;
  ctx.slot_io = ctx.step % p.n_steps;
  const int epoch = *p.epoch;
  ctx.parity = (unsigned)epoch & 1u;
  ctx.tag = (unsigned)epoch + 1u;
  ctx.n = 0;
  bool ok = true;
  for (int gi = 0; gi < p.n_groups && ok; ++gi) {
    const int k = p.groups[gi].k;
    ok = (k <= 256) ? group_phase<1>(p, smem, misc, ctx, gi) : group_phase<2>(p, smem, misc, ctx, gi);
  }
  // Every CTA read the counters at its start and has since taken part in the
  // last group's exchange, so they may advance now.
  if (blockIdx.x == 0 && threadIdx.x == 0 && ok) {
    *p.epoch = epoch + 1;
    if (p.use_counter) *p.step = ctx.step + 1;
  }
}

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
  consumer(p, smem, misc);
}

__global__ void k_abs_max_bf16(const uint16_t* __restrict__ p, size_t n, float* out) {
  // max |P|, written as a float; the values are non-negative so the integer
  // ordering of their bit patterns is the numeric ordering.
  float m = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x) {
    const float v = fabsf(__uint_as_float(((uint32_t)p[i]) << 16));
    m = fmaxf(m, v);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
}

}  // namespace

int persist_smem_bytes() { return kSmemBytes; }
int persist_threads() { return kThreadsP; }

cudaError_t launch_abs_max_bf16(const void* p, size_t n, float* out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
  if (e != cudaSuccess) return e;
  k_abs_max_bf16<<<64, 256, 0, st>>>(static_cast<const uint16_t*>(p), n, out);
  return cudaGetLastError();
}

cudaError_t launch_decode_step(const PersistParams& p, int grid, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_step, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  PersistParams pp = p;
  void* args[] = {&pp};
  // cooperative launch: all CTAs are guaranteed co-resident, which the
  // cross-CTA exchanges rely on
  return cudaLaunchCooperativeKernel((void*)k_decode_step, dim3(grid), dim3(kThreadsP), args,
                                     kSmemBytes, st);
}

}  // namespace gsi
