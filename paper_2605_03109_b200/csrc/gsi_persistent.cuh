// Descriptors of the persistent decode-step kernel (device-resident tables).
#pragma once

#include "gsi_common.cuh"

namespace gsi {

constexpr int kPersistConsumerWarps = 15;  // + 1 producer warp = 16 warps: registers are allotted per 4 warps
constexpr int kPersistMaxPRows = 256;   // basis rows one CTA may own
constexpr int kPersistMaxORows = 512;   // output rows one CTA may own
constexpr int kPersistMaxGrid = 256;    // CTAs (exchange-2 slots per group)
constexpr int kPersistMaxTokens = 2;    // tokens per step served by one launch per token (more: batched kernels)
constexpr int kAccStride = 16;          // 64-bit words between c accumulators: one per 128-byte line

struct PersistGroup {
  const uint16_t* P;                 // [d][k] bf16
  const uint16_t* WP;                // [O][k] bf16, images of all maps concatenated
  const uint16_t* W[GSI_MAX_MAPS];   // [d_out_j][d] bf16
  int off[GSI_MAX_MAPS + 1];
  int n_maps;
  int d, k, O;
  float eps;
  unsigned flags;
  float pmax;                        // max |P| (patched in on the device at bind time)
  const float* x;                    // [n_steps][tokens][d]
  float* y;                          // [tokens][O]
  float* r;                          // [d]
  unsigned long long* acc_c;         // [2][k][kAccStride] fixed-point accumulators, one set per launch parity
  unsigned long long* slot_r;        // exchange 2: 32-bit words [grid + 2] (launch parity in the sign bit | partial ||r||^2)
  unsigned* bar;                     // [6] arrival counters by launch parity: [0..1] after, [2..3] before the gated residual, [4..5] exchange 2
  int p_rows, o_rows;                // rows per CTA of P and of the images (ceil(rows / ncta))
  long long x_step_stride;
  // Two consecutive groups whose inputs do not depend on each other's outputs may form one
  // phase: CTAs [cta0, cta0 + ncta) run this group's projection, gate and image while the
  // rest of the grid runs its partner's; both gates come out of one joint exchange, and a
  // gated residual always streams W with the whole grid.
  int cta0, ncta;                    // this group's share of the grid (0, grid when alone)
  int phase_len;                     // groups in this group's phase: 1, or 2 for both of a pair
  int next_len;                      // groups in the phase after this group's (0 at the end)
  int o_rows_w;                      // W rows per CTA of the gated residual: ceil(O / grid)
};

constexpr int kPairSumSlot = 254;    // pairs need grid + 2 exchange-2 words in 256: word grid + u is ||x||^2 of group u of a pair

struct PersistParams {
  const PersistGroup* groups;  // device
  int n_groups;
  int* step;                   // device: decode-step counter (selects the I/O slot)
  int* epoch;                  // device: launches so far (parity of the exchange buffers)
  int n_steps;
  int use_counter;             // 0: I/O slot 0, counter not advanced
  int n_tokens, token;         // tokens per step, and the one this launch processes (one launch per token)
  int advance;                 // this launch advances the step counter (the last token's launch)
  unsigned char* gate_log;     // [n_steps][n_groups]
  float* rho_log;              // same shape or nullptr
  int log_step_stride;
  int* status;
  unsigned long long* trace;   // device [16] cycle counters of CTA 0, or nullptr
};

int persist_smem_bytes();
int persist_threads();
// pairs: some phase of the table holds two groups; common_k: the rank shared by every gated
// group of the table, or 0 (both select a build of the kernel)
cudaError_t launch_decode_step(const PersistParams& p, int grid, bool pairs, int common_k,
                               cudaStream_t st);
cudaError_t launch_abs_max_bf16(const void* p, size_t n, float* out, cudaStream_t st);
cudaError_t launch_patch_pmax(PersistGroup* groups, const float* const* pmax_ptrs, int n,
                              cudaStream_t st);

}  // namespace gsi
