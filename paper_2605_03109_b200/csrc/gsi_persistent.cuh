// Descriptors of the persistent decode-step kernel (device-resident tables).
#pragma once

#include "gsi_common.cuh"

namespace gsi {

constexpr int kPersistConsumerWarps = 15;  // + 1 producer warp = 16 warps: registers are allotted per 4 warps
constexpr int kPersistMaxPRows = 256;   // basis rows one CTA may own
constexpr int kPersistMaxORows = 512;   // output rows one CTA may own
constexpr int kPersistMaxGrid = 160;    // CTAs (tagged words per group)
constexpr int kPersistMaxTokens = 2;    // tokens per step served by one launch per token (more: batched kernels)
constexpr int kPersistMaxTicks = 160;   // phases of one launch + 2 (the per-CTA plan of a launch lives in shared memory)
constexpr int kPersistPieceBytes = 32768;   // largest contiguous piece of the W stream
constexpr int kPersistMaxD = 16384;     // widest input: a row of W fits one piece, a lane's share of r fits its registers
constexpr int kPersistMaxWRows = 256;   // rows of W (all maps of a group) one CTA may own

// Bytes of 16 rows of a tiled matrix of rank k.
__host__ __device__ inline int persist_image_row_bytes(int k, bool fp8) { return fp8 ? k * 16 + 64 : k * 32; }

struct PersistGroup {
  // Basis [d][k] and concatenated images [O][k], bf16, as 16 x 16 tiles: tile (R, K) at
  // ((R * k/16 + K) * 512) bytes; its 16-byte word l = 4g + t holds elements (g, 2t..2t+1),
  // (g+8, 2t..2t+1), (g, 2t+8..2t+9), (g+8, 2t+8..2t+9): the A operand of mma.m16n8k16.
  // Rows past d (O) are zero.  With GSI_FLAG_FP8_IMAGE the image holds one byte (an E4M3
  // code) per element in the same order (tiles of 256 bytes), and every 16 rows end with
  // their 16 fp32 row scales: persist_image_row_bytes(k, true) bytes per 16 rows.
  const uint16_t* P;
  const uint16_t* WP;
  const uint16_t* W[GSI_MAX_MAPS];   // [d_out_j][d] bf16
  const float* x;                    // [n_steps][tokens][d]
  float* y;                          // [tokens][O]
  float* r;                          // [d]
  // Cross-CTA state.  acc: per launch parity k + 4 contiguous 64-bit fixed-point accumulators
  // whose upper bits count arrivals: c_0..c_{k-1}, ||x||^2, a spare, ||r||^2, a spare (every
  // CTA adds its k + 2 leading words with ONE bulk reduction).  xmax: one 32-bit word per
  // contributing CTA, max |x| over its rows with the launch parity in the sign bit.  pub:
  // ||x||^2 as a double with the launch parity in the sign bit.
  unsigned long long* acc;
  unsigned* xmax;
  unsigned long long* pub;
  unsigned* bar;                     // arrival counters by launch parity: [0..1] after a dense group, [2..3] before a gated residual
  long long x_step_stride;
  int off[GSI_MAX_MAPS + 1];
  int n_maps;
  int d, k, O;
  float eps;
  unsigned flags;
  float pmax;                        // max |P| (patched in on the device at bind time)
  int p_rows, o_rows;                // most rows one CTA owns of P and of the images (multiples of 16)
  int n_contrib;                     // CTAs that own basis rows: the first min(ncta, ceil(d / 16)) of the share
  // Two consecutive groups whose inputs do not depend on each other's outputs may form one
  // phase: CTAs [cta0, cta0 + ncta) run this group's projection, residual and image while the
  // rest of the grid runs its partner's.  A gated residual always streams W with the whole grid.
  int cta0, ncta;                    // this group's share of the grid (0, grid when alone)
  int phase_len;                     // groups in this group's phase: 1, or 2 for both of a pair
  int next_len;                      // groups in the phase after this group's (0 at the end)
  // W stream (gated residual, dense baseline): every CTA owns w_rows[j] consecutive rows of
  // every map j (one contiguous run of memory), copied as contiguous pieces of w_pr whole rows
  // (at most 32 KB).
  short w_rows[GSI_MAX_MAPS];
  int w_pr;
};

struct PersistParams {
  const PersistGroup* groups;  // device
  int n_groups;
  const int* phase_first;      // device [n_phases]: first group of every phase
  int n_phases;
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
  unsigned long long* trace;   // device [grid][16] cycle counters per CTA, or nullptr
  unsigned spin_limit;         // polls a cross-CTA wait may take before it gives up
};

constexpr unsigned kPersistSpinLimitDefault = 1u << 22;

int persist_smem_bytes();
int persist_threads();
// pairs: some phase of the table holds two groups; common_k: the rank shared by every gated
// group of the table, or 0 (both select a build of the kernel)
cudaError_t launch_decode_step(const PersistParams& p, int grid, bool pairs, int common_k,
                               cudaStream_t st);
cudaError_t launch_abs_max_bf16(const void* p, size_t n, float* out, cudaStream_t st);
// Row-major [rows][k] bf16 -> the tiled layout described at PersistGroup::P.
cudaError_t launch_pack_t16(const void* src, int rows, int k, void* dst, cudaStream_t st);
// Row-major [rows][k] bf16 -> E4M3 codes with per-row scales, tiled (see PersistGroup::P).
cudaError_t launch_pack_t16_fp8(const void* src, int rows, int k, void* dst, cudaStream_t st);
cudaError_t launch_patch_pmax(PersistGroup* groups, const float* const* pmax_ptrs, int n,
                              cudaStream_t st);

}  // namespace gsi
