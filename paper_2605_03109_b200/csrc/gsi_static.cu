// gsi_forward_static: the gated subspace layer for callers that cannot allocate.
//
// Every other forward entry point works out of a caller-allocated workspace.
// Some callers have no allocator to hand: code running inside a CUDA-graph
// capture set up by someone else, a plugin loaded into a host program that owns
// all device memory, an interrupt-style hot path that must not touch
// cudaMalloc.  For them the scratch of one small call lives in a fixed array
// compiled into the library.  Every GPU that loads the library holds that array
// (kStaticScratchBytes) until the process exits.
#include "gsi_common.cuh"

namespace {

constexpr int kStaticMaxTokens = 4;
constexpr int kStaticMaxK = 512;
constexpr int kStaticMaxD = 16384;
constexpr int kStaticMaxSlabs = 148;
constexpr int kMaxDevices = 64;

// layout of the scratch array (bytes, each block 256-aligned)
constexpr size_t kOffCtrl = 0;                                                    // 256 B
constexpr size_t kOffFired = 256;                                                 // 256 B
constexpr size_t kOffRho = 512;                                                   // 256 B
constexpr size_t kOffC = 768;                                                     // tokens*k floats
constexpr size_t kOffNorm = kOffC + (size_t)kStaticMaxTokens * kStaticMaxK * 4;
constexpr size_t kOffR = kOffNorm + 8192;
constexpr size_t kOffCpart = kOffR + (size_t)kStaticMaxTokens * kStaticMaxD * 4;
constexpr size_t kStaticScratchBytes =
    kOffCpart + (size_t)kStaticMaxSlabs * kStaticMaxTokens * kStaticMaxK * 4;
static_assert((size_t)kStaticMaxSlabs * kStaticMaxTokens * 2 * 4 <= 8192, "norm partials");
static_assert(kOffNorm % 256 == 0 && kOffR % 256 == 0 && kOffCpart % 256 == 0, "alignment");

// The scratch itself.  In host code this name is only a stand-in for the
// symbol: it is NOT a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the array on each device, resolved once per device.
unsigned char* g_scratch_ptr[kMaxDevices] = {};

gsi_status_t scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return GSI_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return GSI_ERR_UNSUPPORTED;
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    // set-up, once per device, with that device current
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return GSI_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return GSI_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" gsi_status_t gsi_forward_static(const void* const* W_host_array, const int* d_out,
                                           int n_maps, const void* P, gsi_dtype_t p_dtype,
                                           const void* W_P, int d, int k, float eps,
                                           const float* x, int n_tokens, float* y,
                                           unsigned char* gate_mask_out, float* rho_out,
                                           gsi_stream_t stream) {
  using namespace gsi;
  if (!W_host_array || !d_out || !P || !W_P || n_maps <= 0 || d <= 0 || k <= 0 || n_tokens < 0)
    return GSI_ERR_INVALID_ARG;
  if (p_dtype != GSI_BF16 && p_dtype != GSI_F32) return GSI_ERR_INVALID_ARG;
  if (!(eps >= 0.f)) return GSI_ERR_INVALID_ARG;
  // sizes beyond what the built-in scratch holds are refused, never truncated
  if (n_maps > GSI_MAX_MAPS || n_tokens > kStaticMaxTokens || k > kStaticMaxK || d > kStaticMaxD)
    return GSI_ERR_UNSUPPORTED;
  if (d % 8 || k % 8 || k > d) return GSI_ERR_UNSUPPORTED;
  if (n_tokens == 0) return GSI_OK;
  if (!x || !y || !gate_mask_out) return GSI_ERR_INVALID_ARG;
  if (!aligned16(P) || !aligned16(W_P) || !aligned16(x) || !aligned16(y))
    return GSI_ERR_INVALID_ARG;

  GroupParams g{};
  g.d = d;
  g.k = k;
  g.B = n_tokens;
  g.p_f32 = p_dtype == GSI_F32;
  g.eps = eps;
  g.flags = GSI_FLAG_NONE;
  g.P = P;
  g.WP = static_cast<const uint16_t*>(W_P);
  g.n_maps = n_maps;
  int off = 0;
  for (int j = 0; j < n_maps; ++j) {
    if (!W_host_array[j] || !aligned16(W_host_array[j]) || d_out[j] <= 0)
      return GSI_ERR_INVALID_ARG;
    if (d_out[j] % 8) return GSI_ERR_UNSUPPORTED;
    g.W[j] = static_cast<const uint16_t*>(W_host_array[j]);
    g.d_out[j] = d_out[j];
    g.off[j] = off;
    off += d_out[j];
  }
  g.off[n_maps] = off;
  g.O = off;
  int slab = (d + kStaticMaxSlabs - 1) / kStaticMaxSlabs;
  if (slab < 8) slab = 8;
  g.slab_rows = slab;
  g.n_slabs = (d + slab - 1) / slab;

  unsigned char* base = nullptr;
  gsi_status_t st = scratch_for_current_device(&base);
  if (st != GSI_OK) return st;
  int* ctrl = reinterpret_cast<int*>(base + kOffCtrl);
  g.n_fired = ctrl + 0;
  g.counter = reinterpret_cast<unsigned*>(ctrl + 1);
  g.status = ctrl + 2;
  g.fired = reinterpret_cast<int*>(base + kOffFired);
  g.rho_scratch = reinterpret_cast<float*>(base + kOffRho);
  g.c = reinterpret_cast<float*>(base + kOffC);
  g.normpart = reinterpret_cast<float*>(base + kOffNorm);
  g.r = reinterpret_cast<float*>(base + kOffR);
  g.cpart = reinterpret_cast<float*>(base + kOffCpart);

  // The array keeps whatever the last call left.  The arrival counter and the
  // fired count must start at zero; everything else is written before it is read.
  if (cudaMemsetAsync(ctrl, 0, 256, stream) != cudaSuccess) return GSI_ERR_CUDA;

  IoRef io{};
  io.x = x;
  io.y = y;
  io.gate = gate_mask_out;
  io.rho = rho_out;
  io.step = nullptr;
  io.n_steps = 1;
  return launch_generic_forward(g, nullptr, io, n_tokens, stream, nullptr) == cudaSuccess ? GSI_OK
                                                                                  : GSI_ERR_CUDA;
}
