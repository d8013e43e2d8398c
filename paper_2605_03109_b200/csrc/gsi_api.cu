// C ABI of the gated subspace layer: argument checking, workspace layout,
// handle and stack bookkeeping, kernel sequencing.  No arithmetic lives here.
#include <algorithm>
#include <new>
#include <vector>
#include <cstring>

#include "gsi_common.cuh"
#include "gsi_umma.cuh"
#include "gsi_persistent.cuh"

using namespace gsi;

namespace {

constexpr size_t kAlign = 256;
constexpr int kSlabTarget = 148;  // one basis slab per SM of a B200

inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Layout {
  size_t wp, c, cpart, r, normpart, ctrl, fired, rho, x_stage, y_stage, gate_stage, rho_stage,
      pk_acc, pk_slot, tc_rb, tc_ypart, f_pt, f_xb, f_cb, f_cpart, f_normpart, pk_pp, pk_wpp, total;
  int O, n_slabs, slab_rows;
  bool tc, front, dense_tc, packed;
};

constexpr int kTcMinFired = 5;  // fewer fired tokens: one pass of the CUDA-core GEMV
constexpr int kFrontMinTokens = 2;  // single-token calls: the CUDA-core front end

bool tc_shapes_ok(const gsi_desc_t* d) {
  for (int j = 0; j < d->n_maps; ++j)
    if (d->d_out[j] % 128) return false;
  return true;
}

gsi_status_t check_desc(const gsi_desc_t* d) {
  if (!d || !d->d_out) return GSI_ERR_INVALID_ARG;
  if (d->d <= 0 || d->n_maps <= 0 || d->max_tokens <= 0) return GSI_ERR_INVALID_ARG;
  if (d->n_maps > GSI_MAX_MAPS || d->max_tokens > GSI_MAX_TOKENS) return GSI_ERR_UNSUPPORTED;
  if (d->p_dtype != GSI_BF16 && d->p_dtype != GSI_F32) return GSI_ERR_INVALID_ARG;
  if (d->d % 8) return GSI_ERR_UNSUPPORTED;
  for (int j = 0; j < d->n_maps; ++j) {
    if (d->d_out[j] <= 0) return GSI_ERR_INVALID_ARG;
    if (d->d_out[j] % 8) return GSI_ERR_UNSUPPORTED;
  }
  if ((d->flags & GSI_FLAG_FP8_IMAGE) && (d->flags & GSI_FLAG_DENSE)) return GSI_ERR_INVALID_ARG;
  if (!(d->flags & GSI_FLAG_DENSE)) {
    if (d->k <= 0) return GSI_ERR_INVALID_ARG;
    if (d->k % 8 || d->k > 1024 || d->k > d->d) return GSI_ERR_UNSUPPORTED;
    if (!(d->eps >= 0.f)) return GSI_ERR_INVALID_ARG;  // also rejects NaN
  }
  return GSI_OK;
}

Layout make_layout_ws(const gsi_desc_t* d) {
  Layout L{};
  const bool dense = d->flags & GSI_FLAG_DENSE;
  const size_t B = d->max_tokens, k = dense ? 0 : d->k;
  int O = 0;
  for (int j = 0; j < d->n_maps; ++j) O += d->d_out[j];
  L.O = O;
  int slab = (d->d + kSlabTarget - 1) / kSlabTarget;
  if (slab < 8) slab = 8;
  L.slab_rows = slab;
  L.n_slabs = (d->d + slab - 1) / slab;
  size_t at = 0;
  auto take = [&](size_t bytes) { size_t o = at; at += align_up(bytes); return o; };
  L.wp = take((size_t)O * k * 2);
  L.c = take(B * k * 4);
  L.cpart = take((size_t)L.n_slabs * B * k * 4);
  L.r = take(dense ? 0 : B * d->d * 4);
  L.normpart = take((size_t)L.n_slabs * B * 2 * 4);
  L.ctrl = take(256);
  L.fired = take(B * 4);
  L.rho = take(B * 4);
  L.x_stage = take(B * d->d * 4);
  L.y_stage = take(B * (size_t)O * 4);
  L.gate_stage = take(B);
  L.rho_stage = take(B * 4);
  L.pk_acc = take(2 * (k + 4) * 8);                 // persistent kernel: accumulators of c, ||x||^2, ||r||^2
  L.pk_slot = take((size_t)kPersistMaxGrid * 8);    // persistent kernel: tagged max|x| words, published ||x||^2
  // tensor-core kernels: batched handles only
  const bool tc_any = d->max_tokens >= kFrontMinTokens && d->d % 64 == 0 && tc_shapes_ok(d);
  const bool tc = !dense && tc_any;
  const bool dense_tc = dense && tc_any;   // the dense baseline of batched calls, same tile routine
  L.tc_rb = take(tc_any ? (size_t)65 * d->d * 2 : 0);   // row 64 stays zero
  L.tc_ypart = take(tc_any ? (size_t)tc_splits(O, d->d) * 64 * O * 4 : 0);
  L.tc = tc;
  L.dense_tc = dense_tc;
  // tensor-core projection / residual / image for batched calls
  const bool front = tc && d->max_tokens >= kFrontMinTokens && d->p_dtype == GSI_BF16 && d->k % 128 == 0 &&
                     d->d % 128 == 0 && O % 128 == 0;
  const size_t rows = front ? front_rows(d->max_tokens) : 0;
  L.f_pt = take(front ? (size_t)d->k * d->d * 2 : 0);
  L.f_xb = take(rows * d->d * 2);
  L.f_cb = take(rows * k * 2);
  L.f_cpart = take(front ? (size_t)front_proj_splits(d->d, d->k) * B * k * 4 : 0);
  L.f_normpart = take(front ? (size_t)(d->d / 128) * B * 2 * 4 : 0);
  L.front = front;
  // persistent kernel: the basis and the images once more, as 16 x 16 tiles in the operand
  // order of the tensor-core instruction (rows padded to a multiple of 16)
  const bool packed = !dense && d->p_dtype == GSI_BF16 && d->k >= 64 && d->k <= 512 &&
                      (d->k & (d->k - 1)) == 0 && d->max_tokens <= kPersistMaxTokens;
  L.pk_pp = take(packed ? (size_t)((d->d + 15) / 16 * 16) * k * 2 : 0);
  L.pk_wpp = take(packed ? (size_t)((O + 15) / 16) * persist_image_row_bytes(d->k, d->flags & GSI_FLAG_FP8_IMAGE) : 0);
  L.packed = packed;
  L.total = at;
  return L;
}

}  // namespace

struct gsi_layer {
  gsi_desc_t desc;
  int d_out[GSI_MAX_MAPS];
  Layout lay;
  GroupParams gp;
  TmaMaps tm;          // tensor maps of the tensor-core kernels' operands
  bool has_tm = false;
  char* ws;
  float* pmax;     // device: max |P| (bf16 basis only)
  unsigned* bar;   // device: [2] barrier counters of the persistent kernel
  cudaStream_t last_stream;
};

struct gsi_stack {
  int mode;                 // 0 auto, 1 generic kernels, 2 persistent kernel required
  bool persistent;          // the persistent kernel is in use
  int grid;                 // CTAs of the persistent kernel (= SMs)
  bool has_pairs;           // some phase of the persistent schedule holds two groups
  int common_k;             // rank shared by every gated group of the persistent schedule, or 0
  PersistGroup* dev_groups; // device table
  int* dev_phase_first;     // device: first group of every phase of the persistent schedule
  int n_phases;
  std::vector<int> host_phase_first;
  unsigned spin_limit;      // polls a cross-CTA wait of the persistent kernel may take
  std::vector<PersistGroup> host_groups;
  std::vector<const float*> host_pmax_ptrs;
  int* epoch;               // device
  int* status;              // device
  unsigned long long* trace; // device, optional
  std::vector<gsi_layer*> groups;
  std::vector<char> pair_first;   // group i and i+1 declared independent of each other
  std::vector<gsi_stack_io_t> io;
  int B;
  int n_steps;
  unsigned char* gate_log;
  float* rho_log;
  int* step;  // device
  bool bound;
  int seek_value;
  cudaStream_t last_stream;
  // per-stage / batched path: the second group of a concurrent pair runs on a stream of
  // the stack's own, forked from and joined to the caller's stream by events
  cudaStream_t aux = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // batched steps: the chains of small kernels (projection, residual, gate, image) run on a
  // stream of the stack's own with the highest priority, the gated-residual contractions stay
  // on the caller's stream: a contraction is ordered behind its group's gate by an event and
  // runs beside the chains of the groups that follow (inputs are staged before the step)
  cudaStream_t front_stream = nullptr;
  cudaEvent_t ev_resid = nullptr, ev_front_fork = nullptr, ev_front_join = nullptr;
  ~gsi_stack() {
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ev_join) cudaEventDestroy(ev_join);
    if (aux) cudaStreamDestroy(aux);
    if (ev_resid) cudaEventDestroy(ev_resid);
    if (ev_front_fork) cudaEventDestroy(ev_front_fork);
    if (ev_front_join) cudaEventDestroy(ev_front_join);
    if (front_stream) cudaStreamDestroy(front_stream);
  }
};

// The tiled copies of the basis and of the images that the persistent kernel streams.
static bool repack(gsi_layer* h, cudaStream_t stream) {
  const Layout& L = h->lay;
  if (launch_pack_t16(h->gp.P, h->desc.d, h->desc.k, h->ws + L.pk_pp, stream) != cudaSuccess) return false;
  return ((h->desc.flags & GSI_FLAG_FP8_IMAGE)
              ? launch_pack_t16_fp8(h->ws + L.wp, L.O, h->desc.k, h->ws + L.pk_wpp, stream)
              : launch_pack_t16(h->ws + L.wp, L.O, h->desc.k, h->ws + L.pk_wpp, stream)) == cudaSuccess;
}

extern "C" {

const char* gsi_status_string(gsi_status_t s) {
  switch (s) {
    case GSI_OK: return "ok";
    case GSI_ERR_INVALID_ARG: return "invalid argument";
    case GSI_ERR_UNSUPPORTED: return "unsupported shape";
    case GSI_ERR_ALLOC: return "host allocation failed";
    case GSI_ERR_CUDA: return "CUDA runtime error";
    case GSI_ERR_TIMEOUT: return "device-side wait timed out";
    case GSI_ERR_WORKSPACE: return "workspace too small";
  }
  return "unknown status";
}

gsi_status_t gsi_build_image(const void* W, const void* P, int o, int d, int k,
                             gsi_dtype_t p_dtype, void* W_P_out, gsi_stream_t stream) {
  if (!W || !P || !W_P_out || o <= 0 || d <= 0 || k <= 0) return GSI_ERR_INVALID_ARG;
  if (p_dtype != GSI_BF16 && p_dtype != GSI_F32) return GSI_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(P) || !aligned16(W_P_out)) return GSI_ERR_INVALID_ARG;
  if (o % 8 || d % 8 || k % 8) return GSI_ERR_UNSUPPORTED;
  return launch_build_image(W, P, o, d, k, p_dtype == GSI_F32, W_P_out, stream) == cudaSuccess
             ? GSI_OK
             : GSI_ERR_CUDA;
}

size_t gsi_workspace_bytes(const gsi_desc_t* desc) {
  if (check_desc(desc) != GSI_OK) return 0;
  return make_layout_ws(desc).total;
}

gsi_status_t gsi_create(const gsi_desc_t* desc, const void* const* W, const void* P,
                        void* workspace, size_t workspace_bytes, gsi_stream_t stream,
                        gsi_handle_t* out) {
  if (!out) return GSI_ERR_INVALID_ARG;
  *out = nullptr;
  gsi_status_t st = check_desc(desc);
  if (st != GSI_OK) return st;
  const bool dense = desc->flags & GSI_FLAG_DENSE;
  if (!W || !workspace || (!dense && !P)) return GSI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) % kAlign) || (P && !aligned16(P)))
    return GSI_ERR_INVALID_ARG;
  for (int j = 0; j < desc->n_maps; ++j)
    if (!W[j] || !aligned16(W[j])) return GSI_ERR_INVALID_ARG;
  Layout L = make_layout_ws(desc);
  if ((desc->flags & GSI_FLAG_FP8_IMAGE) && !L.packed) return GSI_ERR_UNSUPPORTED;   // the persistent kernel alone reads FP8 images
  if (workspace_bytes < L.total) return GSI_ERR_WORKSPACE;

  gsi_layer* h = new (std::nothrow) gsi_layer();
  if (!h) return GSI_ERR_ALLOC;
  h->desc = *desc;
  std::memcpy(h->d_out, desc->d_out, sizeof(int) * desc->n_maps);
  h->desc.d_out = h->d_out;
  h->lay = L;
  h->ws = static_cast<char*>(workspace);
  h->last_stream = stream;

  GroupParams& g = h->gp;
  std::memset(&g, 0, sizeof g);
  g.d = desc->d;
  g.k = dense ? 8 : desc->k;
  g.O = L.O;
  g.B = desc->max_tokens;
  g.p_f32 = desc->p_dtype == GSI_F32;
  g.eps = desc->eps;
  g.flags = desc->flags;
  g.P = P;
  g.WP = reinterpret_cast<const uint16_t*>(h->ws + L.wp);
  g.n_maps = desc->n_maps;
  int off = 0;
  for (int j = 0; j < desc->n_maps; ++j) {
    g.W[j] = static_cast<const uint16_t*>(W[j]);
    g.d_out[j] = desc->d_out[j];
    g.off[j] = off;
    off += desc->d_out[j];
  }
  g.off[desc->n_maps] = off;
  g.c = reinterpret_cast<float*>(h->ws + L.c);
  g.cpart = reinterpret_cast<float*>(h->ws + L.cpart);
  g.r = reinterpret_cast<float*>(h->ws + L.r);
  g.normpart = reinterpret_cast<float*>(h->ws + L.normpart);
  int* ctrl = reinterpret_cast<int*>(h->ws + L.ctrl);
  g.n_fired = ctrl + 0;
  g.counter = reinterpret_cast<unsigned*>(ctrl + 1);
  g.status = ctrl + 2;
  g.fired = reinterpret_cast<int*>(h->ws + L.fired);
  g.rho_scratch = reinterpret_cast<float*>(h->ws + L.rho);
  g.n_slabs = L.n_slabs;
  g.slab_rows = L.slab_rows;
  g.tc_min_fired = L.tc ? kTcMinFired : 0;
  g.rb = reinterpret_cast<uint16_t*>(h->ws + L.tc_rb);
  g.ypart = reinterpret_cast<float*>(h->ws + L.tc_ypart);
  g.front_min_tokens = (L.front || L.dense_tc) ? kFrontMinTokens : 0;
  g.proj_splits = L.front ? front_proj_splits(desc->d, desc->k) : 0;
  g.PT = reinterpret_cast<const uint16_t*>(h->ws + L.f_pt);
  g.xb = reinterpret_cast<uint16_t*>(h->ws + L.f_xb);
  g.cb = reinterpret_cast<uint16_t*>(h->ws + L.f_cb);
  g.cpart3 = reinterpret_cast<float*>(h->ws + L.f_cpart);
  g.normpart3 = reinterpret_cast<float*>(h->ws + L.f_normpart);

  if (L.tc || L.dense_tc) {
    if (!build_tma_maps(g, L.front, desc->max_tokens, &h->tm)) {
      delete h;
      return GSI_ERR_CUDA;
    }
    h->has_tm = true;
  }

  if (cudaMemsetAsync(ctrl, 0, 256, stream) != cudaSuccess ||
      cudaMemsetAsync(h->ws + L.pk_acc, 0, L.total - L.pk_acc, stream) != cudaSuccess) {
    delete h;
    return GSI_ERR_CUDA;
  }
  h->pmax = reinterpret_cast<float*>(ctrl + 8);
  h->bar = reinterpret_cast<unsigned*>(ctrl + 16);
  if (!dense && !g.p_f32 &&
      launch_abs_max_bf16(P, (size_t)desc->d * desc->k, h->pmax, stream) != cudaSuccess) {
    delete h;
    return GSI_ERR_CUDA;
  }
  if (L.front &&
      launch_transpose_bf16(P, desc->d, desc->k, h->ws + L.f_pt, stream) != cudaSuccess) {
    delete h;
    return GSI_ERR_CUDA;
  }
  if (!dense) {
    for (int j = 0; j < desc->n_maps; ++j) {
      void* dst = h->ws + L.wp + (size_t)g.off[j] * desc->k * 2;
      if (launch_build_image(W[j], P, desc->d_out[j], desc->d, desc->k, g.p_f32, dst, stream) !=
          cudaSuccess) {
        delete h;
        return GSI_ERR_CUDA;
      }
    }
  }
  if (L.packed && !repack(h, stream)) {
    delete h;
    return GSI_ERR_CUDA;
  }
  // A set-up call: return only when the images, max|P| and the cleared state are in
  // place, so the handle may be used from any stream afterwards.
  if (cudaStreamSynchronize(stream) != cudaSuccess) {
    delete h;
    return GSI_ERR_CUDA;
  }
  *out = h;
  return GSI_OK;
}

gsi_status_t gsi_forward_n(gsi_handle_t h, const float* x, int n_tokens, float* y,
                           unsigned char* gate_mask_out, float* rho_out, gsi_stream_t stream) {
  if (!h || n_tokens < 0 || n_tokens > h->desc.max_tokens) return GSI_ERR_INVALID_ARG;
  if (h->desc.flags & GSI_FLAG_FP8_IMAGE) return GSI_ERR_UNSUPPORTED;   // stacks on the persistent kernel only
  if (n_tokens == 0) return GSI_OK;
  if (!x || !y || !gate_mask_out) return GSI_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y)) return GSI_ERR_INVALID_ARG;
  IoRef io{};
  io.x = x;
  io.y = y;
  io.gate = gate_mask_out;
  io.rho = rho_out;
  io.step = nullptr;
  io.n_steps = 1;
  h->last_stream = stream;
  return launch_generic_forward(h->gp, h->has_tm ? &h->tm : nullptr, io, n_tokens, stream, nullptr) == cudaSuccess ? GSI_OK
                                                                                      : GSI_ERR_CUDA;
}

gsi_status_t gsi_forward(gsi_handle_t h, const float* x, float* y, unsigned char* gate_mask_out,
                         gsi_stream_t stream) {
  if (!h) return GSI_ERR_INVALID_ARG;
  return gsi_forward_n(h, x, h->desc.max_tokens, y, gate_mask_out, nullptr, stream);
}

gsi_status_t gsi_forward_host(gsi_handle_t h, const float* x_host, int n_tokens, float* y_host,
                              unsigned char* gate_mask_host, float* rho_host,
                              gsi_stream_t stream) {
  if (!h || n_tokens < 0 || n_tokens > h->desc.max_tokens) return GSI_ERR_INVALID_ARG;
  if (n_tokens == 0) return GSI_OK;
  if (!x_host || !y_host || !gate_mask_host) return GSI_ERR_INVALID_ARG;
  const Layout& L = h->lay;
  float* xs = reinterpret_cast<float*>(h->ws + L.x_stage);
  float* ys = reinterpret_cast<float*>(h->ws + L.y_stage);
  unsigned char* gs = reinterpret_cast<unsigned char*>(h->ws + L.gate_stage);
  float* rs = reinterpret_cast<float*>(h->ws + L.rho_stage);
  const size_t n = n_tokens;
  if (cudaMemcpyAsync(xs, x_host, n * h->desc.d * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return GSI_ERR_CUDA;
  gsi_status_t st = gsi_forward_n(h, xs, n_tokens, ys, gs, rs, stream);
  if (st != GSI_OK) return st;
  // rows of y are contiguous because the device buffer is [n][O] for any n
  if (cudaMemcpyAsync(y_host, ys, n * L.O * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemcpyAsync(gate_mask_host, gs, n, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return GSI_ERR_CUDA;
  if (rho_host &&
      cudaMemcpyAsync(rho_host, rs, n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return GSI_ERR_CUDA;
  return cudaStreamSynchronize(stream) == cudaSuccess ? GSI_OK : GSI_ERR_CUDA;
}

gsi_status_t gsi_extend_basis(gsi_handle_t h, const float* x, float tau, int* k_active,
                              int* appended_out, float* rho_out, gsi_stream_t stream) {
  if (!h || !x || !k_active || !aligned16(x) || !(tau >= 0.f)) return GSI_ERR_INVALID_ARG;
  if (h->desc.flags & GSI_FLAG_DENSE) return GSI_ERR_UNSUPPORTED;
  const Layout& L = h->lay;
  int* ctrl = reinterpret_cast<int*>(h->ws + L.ctrl);
  ExtendArgs a{};
  a.x = x;
  a.tau = tau;
  a.k_active = k_active;
  a.appended_out = appended_out;
  a.rho_out = rho_out;
  a.y_scratch = reinterpret_cast<float*>(h->ws + L.y_stage);
  a.gate_scratch = reinterpret_cast<unsigned char*>(h->ws + L.gate_stage);
  a.ctrl = ctrl + 24;                                       // words 24..27 of the control block
  a.inv_norm = reinterpret_cast<float*>(ctrl + 28);         // words 28..29
  a.x_scratch = reinterpret_cast<float*>(h->ws + L.x_stage);
  a.pmax = h->gp.p_f32 ? nullptr : h->pmax;
  a.PT = L.front ? const_cast<uint16_t*>(h->gp.PT) : nullptr;
  h->last_stream = stream;
  if (launch_extend_basis(h->gp, a, stream) != cudaSuccess) return GSI_ERR_CUDA;
  if (L.packed && !repack(h, stream)) return GSI_ERR_CUDA;   // the tiled copies follow the new column
  return GSI_OK;
}

gsi_status_t gsi_get_image(gsi_handle_t h, int map, const void** out) {
  if (!h || !out || map < 0 || map >= h->desc.n_maps) return GSI_ERR_INVALID_ARG;
  if (h->desc.flags & GSI_FLAG_DENSE) return GSI_ERR_UNSUPPORTED;
  *out = h->ws + h->lay.wp + (size_t)h->gp.off[map] * h->desc.k * 2;
  return GSI_OK;
}

gsi_status_t gsi_get_image_fp8(gsi_handle_t h, const void** out, size_t* bytes_out) {
  if (!h || !out || !bytes_out) return GSI_ERR_INVALID_ARG;
  if (!(h->desc.flags & GSI_FLAG_FP8_IMAGE)) return GSI_ERR_UNSUPPORTED;
  *out = h->ws + h->lay.pk_wpp;
  *bytes_out = (size_t)((h->lay.O + 15) / 16) * persist_image_row_bytes(h->desc.k, true);
  return GSI_OK;
}

gsi_status_t gsi_get_status(gsi_handle_t h, int* device_status) {
  if (!h || !device_status) return GSI_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return GSI_ERR_CUDA;
  if (cudaMemcpy(device_status, h->gp.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return GSI_ERR_CUDA;
  return GSI_OK;
}

gsi_status_t gsi_destroy(gsi_handle_t h) {
  if (!h) return GSI_ERR_INVALID_ARG;
  delete h;
  return GSI_OK;
}

// ------------------------------------------------------------------ stack
size_t gsi_stack_workspace_bytes(int n_groups) {
  if (n_groups <= 0) return 0;
  static_assert(sizeof(PersistGroup) <= 512, "group descriptor outgrew its slot");
  return align_up(256) + align_up((size_t)n_groups * 512) + align_up((size_t)n_groups * 8) +
         align_up((size_t)n_groups * 4);
}

gsi_status_t gsi_stack_create(int n_groups, const gsi_handle_t* groups, void* workspace,
                              size_t workspace_bytes, gsi_stream_t stream, gsi_stack_t* out) {
  if (!out) return GSI_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_groups <= 0 || !groups || !workspace) return GSI_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSI_ERR_INVALID_ARG;
  if (workspace_bytes < gsi_stack_workspace_bytes(n_groups)) return GSI_ERR_WORKSPACE;
  for (int i = 0; i < n_groups; ++i) {
    if (!groups[i]) return GSI_ERR_INVALID_ARG;
    if (groups[i]->desc.max_tokens != groups[0]->desc.max_tokens) return GSI_ERR_INVALID_ARG;
    // a handle's exchange state and scratch serve one use per step
    for (int j = 0; j < i; ++j)
      if (groups[j] == groups[i]) return GSI_ERR_INVALID_ARG;
  }
  gsi_stack* s = new (std::nothrow) gsi_stack();
  if (!s) return GSI_ERR_ALLOC;
  s->groups.assign(groups, groups + n_groups);
  s->pair_first.assign(n_groups, 0);
  s->io.resize(n_groups);
  s->B = groups[0]->desc.max_tokens;
  s->n_steps = 0;
  s->gate_log = nullptr;
  s->rho_log = nullptr;
  s->step = static_cast<int*>(workspace);
  s->epoch = s->step + 1;
  s->status = s->step + 2;
  s->dev_groups = reinterpret_cast<PersistGroup*>(static_cast<char*>(workspace) + 256);
  s->dev_phase_first = reinterpret_cast<int*>(static_cast<char*>(workspace) + align_up(256) +
                                              align_up((size_t)n_groups * 512) + align_up((size_t)n_groups * 8));
  s->spin_limit = kPersistSpinLimitDefault;
  s->mode = 0;
  s->trace = nullptr;
  s->persistent = false;
  s->grid = 0;
  s->bound = false;
  s->last_stream = stream;
  if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    delete s;
    return GSI_ERR_CUDA;
  }
  *out = s;
  return GSI_OK;
}

// The basis rows and the image rows are dealt to the CTAs of a group's share in units of 16
// rows.  One CTA's share fits its buffers, and the 16 KB chunks of its basis slab, and of its
// image slab, each fit the ring together (pass 1 and the image rows run with every chunk of
// their slab resident; one chunk per lane is waited for).
static bool rows_fit(const gsi_layer* h, int ctas) {
  if (ctas <= 0) return false;
  if ((h->desc.flags & GSI_FLAG_DENSE) || h->desc.k <= 0) return true;
  const int pg = ((h->desc.d + 15) / 16 + ctas - 1) / ctas, og = ((h->lay.O + 15) / 16 + ctas - 1) / ctas;
  if (pg * 16 > kPersistMaxPRows || og * 16 > kPersistMaxORows) return false;
  const int gc = std::max(1, 16384 / (h->desc.k * 32));   // groups per chunk
  return (pg + gc - 1) / gc <= 10 && (og + gc - 1) / gc <= 10;
}

// W stream geometry of a group: whole rows per contiguous piece of at most 32 KB.
static int w_piece_rows(int d) { return std::max(1, kPersistPieceBytes / (d * 2)); }

// A row of W fits a piece, and the per-warp partial results of the W stream hold every row a
// CTA owns of every map of a group.
static bool w_rows_fit(const gsi_layer* h, int grid) {
  if (h->desc.d > kPersistMaxD) return false;
  int total = 0;
  for (int j = 0; j < h->desc.n_maps; ++j) total += (h->d_out[j] + grid - 1) / grid;
  return total <= kPersistMaxWRows;
}

// Can this stack run on the persistent kernel?  (one or two tokens per step, bf16 basis
// with a power-of-two rank up to 512, rows that fit the per-CTA buffers and the ring.)
static bool persistent_eligible(const gsi_stack* s, int grid) {
  if (s->B > kPersistMaxTokens || grid <= 0 || grid > kPersistMaxGrid) return false;
  if ((int)s->groups.size() + 2 > kPersistMaxTicks) return false;   // the launch's plan lives in shared memory
  for (const gsi_layer* h : s->groups) {
    const gsi_desc_t& d = h->desc;
    const bool dense = d.flags & GSI_FLAG_DENSE;
    if (dense && s->B > 1) return false;   // a dense group streams W: once for all tokens (batched GEMM)
    if (d.d % 16) return false;
    if (!rows_fit(h, grid) || !w_rows_fit(h, grid)) return false;
    if (!dense && !h->lay.packed) return false;
  }
  return true;
}

// CTAs given to the first group of a pair: in proportion to the bytes its fast path
// streams, between a quarter and three quarters of the grid; 0 if the rows of either
// group do not fit its share (the pair then runs one group after the other).
static int pair_split(const gsi_layer* a, const gsi_layer* b, int grid) {
  if ((a->desc.flags | b->desc.flags) & GSI_FLAG_DENSE) return 0;
  const double wa = (double)(a->desc.d + a->lay.O) * a->desc.k;
  const double wb = (double)(b->desc.d + b->lay.O) * b->desc.k;
  int na = (int)(grid * wa / (wa + wb) + 0.5);
  na = std::max(grid / 4, std::min(grid - grid / 4, na));
  if (!rows_fit(a, na) || !rows_fit(b, grid - na)) return 0;
  return na;
}

gsi_status_t gsi_stack_set_concurrent(gsi_stack_t s, int first_group, int enable) {
  if (!s || first_group < 0 || first_group + 1 >= (int)s->groups.size()) return GSI_ERR_INVALID_ARG;
  // a group belongs to at most one pair
  if (enable && ((first_group > 0 && s->pair_first[first_group - 1]) || s->pair_first[first_group + 1]))
    return GSI_ERR_INVALID_ARG;
  s->pair_first[first_group] = enable ? 1 : 0;
  s->bound = false;  // applied at bind time
  return GSI_OK;
}

gsi_status_t gsi_stack_set_mode(gsi_stack_t s, int mode) {
  if (!s || mode < 0 || mode > 2) return GSI_ERR_INVALID_ARG;
  s->mode = mode;
  s->bound = false;  // the choice is taken at bind time
  return GSI_OK;
}

gsi_status_t gsi_stack_bind(gsi_stack_t s, const gsi_stack_io_t* io, int n_steps,
                            unsigned char* gate_log, float* rho_log, gsi_stream_t stream) {
  if (!s || !io || n_steps <= 0 || !gate_log) return GSI_ERR_INVALID_ARG;
  const int G = (int)s->groups.size();
  for (int i = 0; i < G; ++i)
    if (!io[i].x || !io[i].y || !aligned16(io[i].x) || !aligned16(io[i].y))
      return GSI_ERR_INVALID_ARG;
  std::copy(io, io + G, s->io.begin());
  s->n_steps = n_steps;
  s->gate_log = gate_log;
  s->rho_log = rho_log;
  s->last_stream = stream;

  s->persistent = false;
  if (s->mode != 1) {
    int dev = 0, sms = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
      return GSI_ERR_CUDA;
    s->grid = sms;
    s->persistent = coop && persistent_eligible(s, sms);
    if (s->mode == 2 && !s->persistent) return GSI_ERR_UNSUPPORTED;
  }
  if (!s->persistent)
    for (const gsi_layer* h : s->groups)
      if (h->desc.flags & GSI_FLAG_FP8_IMAGE) return GSI_ERR_UNSUPPORTED;
  if (!s->persistent && !s->aux) {
    bool any = false;
    for (char c : s->pair_first) any = any || c;
    int least = 0, greatest = 0;
    if (any && (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess ||
                cudaStreamCreateWithPriority(&s->aux, cudaStreamNonBlocking, greatest) != cudaSuccess ||
                cudaEventCreateWithFlags(&s->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&s->ev_join, cudaEventDisableTiming) != cudaSuccess))
      return GSI_ERR_CUDA;
  }
  if (!s->persistent && !s->front_stream) {
    bool any = false;   // some group takes the tensor-core front end at this batch
    for (const gsi_layer* h : s->groups)
      any = any || (h->has_tm && h->gp.front_min_tokens > 0 && s->B >= h->gp.front_min_tokens &&
                    !(h->desc.flags & (GSI_FLAG_DENSE | GSI_FLAG_STATIC_PROJECTION)));
    int least = 0, greatest = 0;
    if (any && (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess ||
                cudaStreamCreateWithPriority(&s->front_stream, cudaStreamNonBlocking, greatest) != cudaSuccess ||
                cudaEventCreateWithFlags(&s->ev_resid, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&s->ev_front_fork, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&s->ev_front_join, cudaEventDisableTiming) != cudaSuccess))
      return GSI_ERR_CUDA;
  }
  if (s->persistent) {
    // The cross-CTA exchange state of every group (accumulators, exchange words, arrival
    // counters) is tied to THIS stack's launch counter: start both from zero.  A handle
    // can therefore serve only one bound stack at a time.
    if (cudaMemsetAsync(s->epoch, 0, sizeof(int), stream) != cudaSuccess ||
        cudaMemsetAsync(s->status, 0, 2 * sizeof(int), stream) != cudaSuccess)   // a fresh start also after a time-out (status word, site of the wait that gave up)
      return GSI_ERR_CUDA;
    for (int i = 0; i < G; ++i) {
      const gsi_layer* h = s->groups[i];
      if (cudaMemsetAsync(h->ws + h->lay.pk_acc, 0, h->lay.tc_rb - h->lay.pk_acc, stream) !=
              cudaSuccess ||
          cudaMemsetAsync(h->bar, 0, 6 * sizeof(unsigned), stream) != cudaSuccess)
        return GSI_ERR_CUDA;
    }
    s->host_groups.assign(G, PersistGroup{});
    s->host_pmax_ptrs.assign(G, nullptr);
    for (int i = 0; i < G; ++i) {
      const gsi_layer* h = s->groups[i];
      PersistGroup& pg = s->host_groups[i];
      const GroupParams& gp = h->gp;
      pg.P = reinterpret_cast<const uint16_t*>(h->ws + h->lay.pk_pp);
      pg.WP = reinterpret_cast<const uint16_t*>(h->ws + h->lay.pk_wpp);
      for (int j = 0; j < gp.n_maps; ++j) {
        pg.W[j] = gp.W[j];
        pg.w_rows[j] = (short)((gp.d_out[j] + s->grid - 1) / s->grid);
      }
      pg.w_pr = w_piece_rows(gp.d);
      for (int j = 0; j <= gp.n_maps; ++j) pg.off[j] = gp.off[j];
      pg.n_maps = gp.n_maps;
      pg.d = gp.d;
      const bool dense_g = gp.flags & GSI_FLAG_DENSE;
      pg.k = dense_g ? 256 : gp.k;
      pg.O = gp.O;
      pg.eps = gp.eps;
      pg.flags = gp.flags;
      pg.pmax = 0.f;
      s->host_pmax_ptrs[i] = (gp.flags & GSI_FLAG_DENSE) ? nullptr : h->pmax;
      pg.x = io[i].x;
      pg.y = io[i].y;
      pg.r = gp.r;
      pg.acc = reinterpret_cast<unsigned long long*>(h->ws + h->lay.pk_acc);
      pg.xmax = reinterpret_cast<unsigned*>(h->ws + h->lay.pk_slot);
      pg.pub = reinterpret_cast<unsigned long long*>(h->ws + h->lay.pk_slot + (size_t)kPersistMaxGrid * 4);
      pg.bar = h->bar;
      pg.cta0 = 0;
      pg.ncta = s->grid;
      pg.phase_len = 1;
      pg.x_step_stride = (long long)s->B * gp.d;
    }
    // pairs of independent groups split the grid
    for (int i = 0; i + 1 < G; ++i) {
      if (!s->pair_first[i]) continue;
      const int na = pair_split(s->groups[i], s->groups[i + 1], s->grid);
      if (na == 0) continue;
      PersistGroup &a = s->host_groups[i], &b = s->host_groups[i + 1];
      a.ncta = na;
      b.cta0 = na;
      b.ncta = s->grid - na;
      a.phase_len = b.phase_len = 2;
    }
    for (int i = 0; i < G; ++i) {
      PersistGroup& pg = s->host_groups[i];
      // rows are dealt in groups of 16: CTA c of the share owns groups [c n / ncta, (c + 1) n / ncta)
      // (the first n CTAs one group each when there are fewer groups than CTAs)
      const int pgroups = (pg.d + 15) / 16, ogroups = (pg.O + 15) / 16;
      pg.p_rows = 16 * ((pgroups + pg.ncta - 1) / pg.ncta);
      pg.o_rows = 16 * ((ogroups + pg.ncta - 1) / pg.ncta);
      pg.n_contrib = std::min(pg.ncta, pgroups);
    }
    s->has_pairs = false;
    s->common_k = -1;
    for (int i = 0; i < G; ++i) {
      if (s->host_groups[i].flags & GSI_FLAG_DENSE) continue;
      const int k = s->host_groups[i].k;
      s->common_k = s->common_k < 0 || s->common_k == k ? k : 0;
    }
    if (s->common_k < 0) s->common_k = 0;
    s->host_phase_first.clear();
    for (int i = 0; i < G;) {   // length of the phase after each group's
      const int len = s->host_groups[i].phase_len;
      s->host_phase_first.push_back(i);
      const int nxt = i + len < G ? s->host_groups[i + len].phase_len : 0;
      for (int j = 0; j < len; ++j) s->host_groups[i + j].next_len = nxt;
      if (len == 2) s->has_pairs = true;
      i += len;
    }
    s->n_phases = (int)s->host_phase_first.size();
    const float** dev_ptrs = reinterpret_cast<const float**>(
        reinterpret_cast<char*>(s->dev_groups) + (size_t)G * 512);
    if (cudaMemcpyAsync(s->dev_groups, s->host_groups.data(), sizeof(PersistGroup) * G,
                        cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dev_ptrs, s->host_pmax_ptrs.data(), sizeof(float*) * G,
                        cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(s->dev_phase_first, s->host_phase_first.data(),
                        s->host_phase_first.size() * sizeof(int), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        launch_patch_pmax(s->dev_groups, dev_ptrs, G, stream) != cudaSuccess)
      return GSI_ERR_CUDA;
  }
  // A set-up call: the descriptor table and the cleared exchange state must be in
  // device memory before a step may be enqueued on ANY stream.
  if (cudaStreamSynchronize(stream) != cudaSuccess) return GSI_ERR_CUDA;
  s->bound = true;
  return GSI_OK;
}

gsi_status_t gsi_stack_seek(gsi_stack_t s, int step, gsi_stream_t stream) {
  if (!s || step < 0) return GSI_ERR_INVALID_ARG;
  s->last_stream = stream;
  s->seek_value = step;  // pageable source: staged by the runtime before the call returns
  return cudaMemcpyAsync(s->step, &s->seek_value, sizeof(int), cudaMemcpyHostToDevice, stream) ==
                 cudaSuccess
             ? GSI_OK
             : GSI_ERR_CUDA;
}

static gsi_status_t stack_enqueue(gsi_stack_t s, bool use_counter, gsi_stream_t stream) {
  const int G = (int)s->groups.size();
  if (s->persistent) {
    PersistParams p{};
    p.groups = s->dev_groups;
    p.n_groups = G;
    p.phase_first = s->dev_phase_first;
    p.n_phases = s->n_phases;
    p.step = s->step;
    p.epoch = s->epoch;
    p.n_steps = s->n_steps;
    p.use_counter = use_counter ? 1 : 0;
    p.gate_log = s->gate_log;
    p.rho_log = s->rho_log;
    p.log_step_stride = G;
    p.status = s->status;
    p.trace = s->trace;
    p.spin_limit = s->spin_limit - 1;   // the kernels give up when a wait has polled more than this many times without success
    p.n_tokens = s->B;
    // one launch per token of the step (up to kPersistMaxTokens; larger batches take the
    // batched kernels): each is a complete decode step of that token, the last one advances
    for (int t = 0; t < s->B; ++t) {
      p.token = t;
      p.advance = t == s->B - 1;
      if (launch_decode_step(p, s->grid, s->has_pairs, s->common_k, stream) != cudaSuccess) return GSI_ERR_CUDA;
    }
    return GSI_OK;
  }
  // fs: the stream the chains of small kernels run on
  cudaStream_t fs = stream;
  ResidualLane lane{stream, s->ev_resid, false};
  if (s->front_stream) {
    if (cudaEventRecord(s->ev_front_fork, stream) != cudaSuccess ||
        cudaStreamWaitEvent(s->front_stream, s->ev_front_fork, 0) != cudaSuccess)
      return GSI_ERR_CUDA;
    fs = s->front_stream;
  }
  auto enqueue_group = [&](int i, cudaStream_t st) -> bool {
    gsi_layer* h = s->groups[i];
    IoRef io{};
    io.x = s->io[i].x;
    io.y = s->io[i].y;
    io.gate = s->gate_log + (size_t)i * s->B;
    io.rho = s->rho_log ? s->rho_log + (size_t)i * s->B : nullptr;
    io.step = use_counter ? s->step : nullptr;
    io.n_steps = s->n_steps;
    io.x_step_stride = (long long)s->B * h->desc.d;
    io.log_step_stride = (long long)G * s->B;
    h->last_stream = stream;   // the joins below put all of the step's work in the caller's stream order
    return launch_generic_forward(h->gp, h->has_tm ? &h->tm : nullptr, io, s->B, st, nullptr,
                                  s->front_stream ? &lane : nullptr) == cudaSuccess;
  };
  for (int i = 0; i < G; ++i) {
    if (s->aux && i + 1 < G && s->pair_first[i]) {
      // groups i and i+1 do not read each other's outputs: two chains of dependent launches
      // side by side (under stream capture this becomes a fork and a join in the graph)
      if (cudaEventRecord(s->ev_fork, fs) != cudaSuccess ||
          cudaStreamWaitEvent(s->aux, s->ev_fork, 0) != cudaSuccess)
        return GSI_ERR_CUDA;
      if (!enqueue_group(i, fs) || !enqueue_group(i + 1, s->aux)) return GSI_ERR_CUDA;
      if (cudaEventRecord(s->ev_join, s->aux) != cudaSuccess ||
          cudaStreamWaitEvent(fs, s->ev_join, 0) != cudaSuccess)
        return GSI_ERR_CUDA;
      ++i;
      continue;
    }
    if (!enqueue_group(i, fs)) return GSI_ERR_CUDA;
  }
  if (s->front_stream &&   // the chains join the caller's stream, which holds the contractions
      (cudaEventRecord(s->ev_front_join, fs) != cudaSuccess ||
       cudaStreamWaitEvent(stream, s->ev_front_join, 0) != cudaSuccess))
    return GSI_ERR_CUDA;
  if (use_counter && launch_advance_step(s->step, stream) != cudaSuccess) return GSI_ERR_CUDA;
  return GSI_OK;
}

gsi_status_t gsi_stack_step(gsi_stack_t s, gsi_stream_t stream) {
  if (!s || !s->bound) return GSI_ERR_INVALID_ARG;
  s->last_stream = stream;
  return stack_enqueue(s, true, stream);
}

gsi_status_t gsi_stack_launches_per_step(gsi_stack_t s, int* n_out) {
  if (!s || !n_out || !s->bound) return GSI_ERR_INVALID_ARG;
  if (s->persistent) {
    *n_out = s->B;
    return GSI_OK;
  }
  int n = 0;
  for (gsi_layer* h : s->groups) {
    n += generic_launch_count(h->gp, s->B);
  }
  *n_out = n + 1;
  return GSI_OK;
}

gsi_status_t gsi_stack_step_host(gsi_stack_t s, const float* const* x_host, float* const* y_host,
                                 unsigned char* gate_host, gsi_stream_t stream) {
  if (!s || !s->bound || !x_host || !y_host || !gate_host) return GSI_ERR_INVALID_ARG;
  const int G = (int)s->groups.size();
  for (int i = 0; i < G; ++i)
    if (!x_host[i] || !y_host[i]) return GSI_ERR_INVALID_ARG;
  // Runs of groups whose buffers are adjacent both on the host and on the device
  // (a caller that carves them out of one arena) travel as ONE copy.
  auto copy_runs = [&](bool to_device) -> bool {
    for (int i = 0; i < G;) {
      const char* h0 = to_device ? reinterpret_cast<const char*>(x_host[i])
                                 : reinterpret_cast<const char*>(y_host[i]);
      const char* d0 = to_device ? reinterpret_cast<const char*>(s->io[i].x)
                                 : reinterpret_cast<const char*>(s->io[i].y);
      size_t bytes = 0;
      int j = i;
      for (; j < G; ++j) {
        const size_t b = to_device ? (size_t)s->B * s->groups[j]->desc.d * 4
                                   : (size_t)s->B * s->groups[j]->lay.O * 4;
        const char* hj = to_device ? reinterpret_cast<const char*>(x_host[j])
                                   : reinterpret_cast<const char*>(y_host[j]);
        const char* dj = to_device ? reinterpret_cast<const char*>(s->io[j].x)
                                   : reinterpret_cast<const char*>(s->io[j].y);
        if (hj != h0 + bytes || dj != d0 + bytes) break;
        bytes += b;
      }
      const cudaError_t e =
          to_device ? cudaMemcpyAsync(const_cast<char*>(d0), h0, bytes, cudaMemcpyHostToDevice, stream)
                    : cudaMemcpyAsync(const_cast<char*>(h0), d0, bytes, cudaMemcpyDeviceToHost, stream);
      if (e != cudaSuccess) return false;
      i = j;
    }
    return true;
  };
  if (!copy_runs(true)) return GSI_ERR_CUDA;
  s->last_stream = stream;
  gsi_status_t st = stack_enqueue(s, false, stream);
  if (st != GSI_OK) return st;
  if (!copy_runs(false)) return GSI_ERR_CUDA;
  if (cudaMemcpyAsync(gate_host, s->gate_log, (size_t)G * s->B, cudaMemcpyDeviceToHost, stream) !=
      cudaSuccess)
    return GSI_ERR_CUDA;
  return cudaStreamSynchronize(stream) == cudaSuccess ? GSI_OK : GSI_ERR_CUDA;
}

gsi_status_t gsi_stack_set_trace(gsi_stack_t s, unsigned long long* cycles) {
  if (!s) return GSI_ERR_INVALID_ARG;
  s->trace = cycles;
  return GSI_OK;
}

gsi_status_t gsi_stack_set_spin_limit(gsi_stack_t s, unsigned polls) {
  if (!s) return GSI_ERR_INVALID_ARG;
  s->spin_limit = polls ? polls : kPersistSpinLimitDefault;
  return GSI_OK;
}

gsi_status_t gsi_stack_is_persistent(gsi_stack_t s, int* out) {
  if (!s || !out || !s->bound) return GSI_ERR_INVALID_ARG;
  *out = s->persistent ? 1 : 0;
  return GSI_OK;
}

gsi_status_t gsi_stack_get_status(gsi_stack_t s, int* device_status) {
  if (!s || !device_status) return GSI_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(s->last_stream) != cudaSuccess) return GSI_ERR_CUDA;
  *device_status = 0;
  if (cudaMemcpy(device_status, s->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return GSI_ERR_CUDA;
  if (*device_status) return GSI_OK;
  for (gsi_layer* h : s->groups) {
    int v = 0;
    if (cudaMemcpy(&v, h->gp.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
      return GSI_ERR_CUDA;
    if (v) {
      *device_status = v;
      break;
    }
  }
  return GSI_OK;
}

gsi_status_t gsi_stack_destroy(gsi_stack_t s) {
  if (!s) return GSI_ERR_INVALID_ARG;
  delete s;
  return GSI_OK;
}

}  // extern "C"
