/*
 * gsi.h - C ABI of the B200 (sm_100a) gated subspace linear layer.
 *
 * The library implements the per-token procedure of Algorithm 1 ("Gated
 * Subspace Inference") for batch-1 and small-batch decode.  For one input
 * activation x (fp32, length d), a stored basis P (d x k; the paper's V_k) and
 * one or more weight matrices W_j (d_out_j x d, bf16) that share this input:
 *
 *   c   = P^T x                          Algorithm 1 line 1 (paper: g = V_k^T x)
 *   r   = x - P c                        line 2, Eq. (3.1); explicit residual
 *   rho = ||r||_2 / ||x||_2              line 3, Eq. (3.3)
 *   y_j = W_P,j c                        line 5; W_P,j = W_j P is the cached
 *                                        image M of Eq. (3.2) / Section 4.2
 *   if !(||r|| < eps ||x||):  y_j += W_j r      Eq. (3.2): y = M g + W r = W x
 *
 * The gate test is the strict comparison of Section 3.2 (fast path iff
 * rho < eps) taken in the division-free form ||r|| < eps*||x||, so x = 0 and
 * non-finite inputs take the slow path.  A token whose gate byte is 1 is
 * "gated" / "fired": the full correction W r was added for it.
 *
 * A "group" is the set of maps sharing one input x (hence one P, c, r and one
 * gate decision per token), e.g. {q, k, v, fc} of a GPT-J block.
 *
 * Conventions
 *   - All pointers are DEVICE pointers unless the name ends in _host.
 *   - Matrices are dense row-major: W [d_out][d], P [d][k], W_P [sum d_out][k].
 *   - bf16 = upper half of IEEE fp32, stored as 16-bit words.
 *   - x is [n_tokens][d] fp32.  y is ONE buffer [n_tokens][sum_j d_out_j] fp32:
 *     token t, map j occupies columns [off_j, off_j + d_out_j), off_j the
 *     running sum of d_out.  y is overwritten, never accumulated into.
 *   - Pointers must be 16-byte aligned; d, k and every d_out multiples of 8;
 *     8 <= k <= min(d, 1024).  Otherwise GSI_ERR_UNSUPPORTED / INVALID_ARG.
 *   - Every function returns gsi_status_t; no exception crosses the boundary.
 *     Argument errors are found on the host before anything is launched.
 *   - Ownership: the caller owns W, P, x, y, the logs and the workspace.  The
 *     library borrows W and P (they must outlive the handle) and owns what it
 *     places in the workspace.  Nothing below allocates device memory.  The
 *     set-up calls (gsi_create, gsi_stack_create, gsi_stack_bind) run their
 *     device work on `stream` and synchronise it before returning, so what they
 *     built may be used from any stream afterwards; they may not be captured.
 *     The forward / step calls do not synchronise the host and may be
 *     stream-captured (the *_host variants copy and synchronise, and may not).
 *   - One handle / stack may be used by one stream at a time.
 */
#ifndef GSI_H_
#define GSI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GSI_OK = 0,
  GSI_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer */
  GSI_ERR_UNSUPPORTED = 2, /* shape outside the supported set                       */
  GSI_ERR_ALLOC = 3,       /* host allocation failed                                */
  GSI_ERR_CUDA = 4,        /* a CUDA runtime call failed                            */
  GSI_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (status word)      */
  GSI_ERR_WORKSPACE = 6    /* workspace smaller than gsi_workspace_bytes()          */
} gsi_status_t;

typedef enum { GSI_BF16 = 0, GSI_F32 = 1 } gsi_dtype_t;

/* A CUDA stream (cudaStream_t), spelt without the CUDA headers. */
typedef struct CUstream_st* gsi_stream_t;

typedef struct gsi_layer* gsi_handle_t; /* one group */
typedef struct gsi_stack* gsi_stack_t;  /* an ordered chain of groups */

enum {
  GSI_FLAG_NONE = 0u,
  /* Static projection (Remark after Theorem 3.1, "Mode C"): never add W r.
     Gate bytes and rho are still reported. */
  GSI_FLAG_STATIC_PROJECTION = 1u,
  /* Dense baseline: y = W x, no projection, no image; gate bytes are written as
     1.  Used to measure the speed-up honestly.  Single-token calls: streaming
     GEMV on the fp32 x.  Calls of 2 or more tokens (d a multiple of 64, every
     d_out a multiple of 128): tensor-core GEMM with x rounded to bf16, as an
     ordinary bf16 GEMM takes its activations. */
  GSI_FLAG_DENSE = 2u,
  /* The image is kept in FP8 (Section 7.4: halves the bytes the fast path
     reads; the paper leaves format and quality open).  Here: E4M3 codes of the
     BF16 image with one fp32 scale per output row, scale = max|row| / 448 (1 for
     a zero row), code = nearest E4M3 (ties to even, saturating) of
     element / scale, both divisions single fp32 operations; y = scale * (codes . c).
     Served by the persistent stack kernel only (bf16 basis, k a power of two in
     64..512, max_tokens <= 2): gsi_create returns GSI_ERR_UNSUPPORTED otherwise,
     and so do the single-group forward calls and binding a stack that cannot run
     persistently.  Not combinable with GSI_FLAG_DENSE. */
  GSI_FLAG_FP8_IMAGE = 4u
};

typedef struct {
  int d;               /* input width                                           */
  int k;               /* basis rank                                            */
  int n_maps;          /* maps sharing this input, 1..GSI_MAX_MAPS              */
  const int* d_out;    /* HOST array [n_maps]                                   */
  float eps;           /* gate threshold: fast path iff ||r|| < eps*||x||       */
  int max_tokens;      /* largest batch a forward call may carry, 1..GSI_MAX_TOKENS */
  gsi_dtype_t p_dtype; /* storage type of P                                     */
  unsigned flags;      /* GSI_FLAG_*                                            */
} gsi_desc_t;

#define GSI_MAX_MAPS 8
#define GSI_MAX_TOKENS 64

const char* gsi_status_string(gsi_status_t s);

/*
 * Cached image of Eq. (3.2) / Section 4.2 (built once per weight matrix, off the per-token path):
 *   W_P[a][j] = bf16_rne( sum_i W[a][i] * P[i][j] ),  fp32 accumulation.
 * W [o][d] bf16, P [d][k] of p_dtype, W_P_out [o][k] bf16; all device.
 * Enqueued on `stream`; no host synchronisation.
 */
gsi_status_t gsi_build_image(const void* W, const void* P, int o, int d, int k,
                             gsi_dtype_t p_dtype, void* W_P_out, gsi_stream_t stream);

/* Bytes of device workspace a handle for `desc` needs (0 if desc is invalid).
 * The workspace holds the images of all maps and the per-call scratch (c, r,
 * partial sums, fired-token list, status word; for max_tokens >= 2 also a
 * transposed copy of the basis and the bf16 operands of the batched kernels). */
size_t gsi_workspace_bytes(const gsi_desc_t* desc);

/*
 * Create a handle for one group.  W_host_array is a HOST array of n_maps DEVICE
 * pointers, W_j [d_out_j][d] bf16.  P is [d][k].  `workspace` is device memory
 * of at least gsi_workspace_bytes(desc), 256-byte aligned, owned by the caller
 * and used exclusively by this handle until gsi_destroy.  The images W_P,j are
 * built on `stream` inside this call (Section 4.2); W is not needed for that
 * again, but is read by every gated token afterwards.
 */
gsi_status_t gsi_create(const gsi_desc_t* desc, const void* const* W_host_array,
                        const void* P, void* workspace, size_t workspace_bytes,
                        gsi_stream_t stream, gsi_handle_t* out);

/*
 * Algorithm 1 for desc.max_tokens tokens (gsi_forward) or n_tokens <=
 * max_tokens tokens (gsi_forward_n).  x [n][d] fp32; y [n][sum d_out] fp32;
 * gate_mask_out [n] bytes (1 = slow path, W r added); rho_out [n] fp32 or NULL.
 * Each token is processed independently of the others in the call (Algorithm 1
 * is per token); its rounding can depend on the size of the call: calls of 2 or
 * more tokens (bf16 basis; k, d and every d_out multiples of 128) run the
 * contractions on the tensor cores with exactly split operands and another
 * summation order and add W r from r rounded to bf16 (|dy| <= 3e-3 max|y|);
 * with other shapes that rounding applies from 5 gated tokens per call on.
 * Results of a given call are reproducible bit for bit.
 * Enqueues on `stream` and returns; n_tokens = 0 is a no-op.
 */
gsi_status_t gsi_forward(gsi_handle_t h, const float* x, float* y,
                         unsigned char* gate_mask_out, gsi_stream_t stream);
gsi_status_t gsi_forward_n(gsi_handle_t h, const float* x, int n_tokens, float* y,
                           unsigned char* gate_mask_out, float* rho_out,
                           gsi_stream_t stream);

/*
 * Same as gsi_forward_n with HOST buffers: copies x to the device, runs the
 * layer, copies y / gate / rho back and synchronises `stream`.  Staging space
 * for x, y, gate and rho is part of the handle's workspace.
 */
gsi_status_t gsi_forward_host(gsi_handle_t h, const float* x_host, int n_tokens,
                              float* y_host, unsigned char* gate_mask_host,
                              float* rho_host, gsi_stream_t stream);

/*
 * The same layer for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant of gsi_forward_n, not a method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin inside
 * a host application that owns all device memory, a library called while
 * someone else's stream capture is open, a latency-critical path that may not
 * enter the allocator.  Such a caller cannot provide the workspace gsi_create
 * wants.  Here the scratch (coefficients, residual, partial sums, fired-token
 * list) lives in a fixed array inside the library: about 1.5 MB that every GPU
 * which loads the library holds until the process exits.  No device status word can
 * be read back for this entry point (its kernels contain no bounded wait).
 *
 * The caller passes everything else: W_host_array (HOST array of n_maps DEVICE
 * pointers, W_j [d_out_j][d] bf16), d_out (HOST array), P [d][k], and W_P, the
 * images of all maps concatenated, [sum d_out][k] bf16, each built once with
 * gsi_build_image (which does not allocate either).  x [n][d], y [n][sum d_out],
 * gate_mask_out [n], rho_out [n] or NULL, as in gsi_forward_n.
 *
 * Limits: n_tokens <= 4, k <= 512, d <= 16384, n_maps <= GSI_MAX_MAPS; larger
 * sizes return GSI_ERR_UNSUPPORTED and nothing is launched.
 *
 * The first call on each device resolves the array's device address (with that
 * device current); make that first call before any stream capture begins.  The
 * call allocates nothing and frees nothing.  All calls on a device share the one
 * array, which keeps the previous call's contents: the counters that must start
 * at zero are cleared on `stream` at the start of every call.  Two calls whose
 * kernels overlap on the GPU (different streams, or one stream per thread) race
 * on the array - serialise them.
 */
gsi_status_t gsi_forward_static(const void* const* W_host_array, const int* d_out, int n_maps,
                                const void* P, gsi_dtype_t p_dtype, const void* W_P, int d,
                                int k, float eps, const float* x, int n_tokens, float* y,
                                unsigned char* gate_mask_out, float* rho_out,
                                gsi_stream_t stream);

/*
 * Online extension of the basis by one vector (the paper's "time-dimension
 * tracking", Section 5.4, and "online basis adaptation", Section 7.2): the token
 * x [d] (fp32, device) is tested against the basis in use; if
 *     rho = ||x - P P^T x|| / ||x||  >  tau
 * and a column is free, the residual orthogonalised against P twice
 * (Gram-Schmidt with one re-orthogonalisation, "DGKS") and normalised is stored,
 * rounded to the basis type, as column *k_active of P, and W times that stored
 * column (Section 4.2), rounded to bf16, as column *k_active of every cached
 * image; *k_active is then incremented.  Layout contract: columns
 * [*k_active, k) of P are zero when the handle is created, so every forward
 * call works on the full width k before and after.
 *
 * This call WRITES the caller's basis buffer P (the pointer given to
 * gsi_create, which must therefore be writable) and the images in the
 * workspace.  k_active: device int, in/out.  appended_out (device int, 0/1) and
 * rho_out (device float) may be NULL.  tau >= 0.  A non-finite token never
 * extends the basis.  Enqueues on `stream` (one pass over W when a column is
 * appended) and returns; it must not overlap a forward call of the same handle,
 * it overwrites the handle's per-call scratch, and a stack that has the handle
 * bound must be bound again afterwards (it caches max|P|).  Not available for
 * GSI_FLAG_DENSE handles.
 */
gsi_status_t gsi_extend_basis(gsi_handle_t h, const float* x, float tau, int* k_active,
                              int* appended_out, float* rho_out, gsi_stream_t stream);

/* Device pointer to the image of map j inside the workspace ([d_out_j][k] bf16),
 * so a caller can inspect or persist it. */
gsi_status_t gsi_get_image(gsi_handle_t h, int map, const void** W_P_out);

/* GSI_FLAG_FP8_IMAGE handles: device pointer to the FP8 image of ALL maps
 * (rows in map order, O = sum d_out, padded with zero rows to a multiple of 16)
 * as the persistent kernel streams it, and its size in bytes.  Per 16 rows R:
 * k/16 tiles of 256 bytes, then the 16 row scales (fp32).  In tile K, the 8
 * bytes at 8*l (l = 4g + t, g < 8, t < 4) are the codes of elements (row, column
 * within the tile) (g,2t) (g,2t+1) (g+8,2t) (g+8,2t+1) (g,2t+8) (g,2t+9)
 * (g+8,2t+8) (g+8,2t+9).  gsi_get_image still returns the BF16 image the codes
 * were taken from. */
gsi_status_t gsi_get_image_fp8(gsi_handle_t h, const void** tiled_out, size_t* bytes_out);

/* Synchronises the handle's last stream and returns the device status word:
 * 0, or a GSI_ERR_* code recorded by a kernel (e.g. a bounded wait that gave
 * up).  Kernels never trap. */
gsi_status_t gsi_get_status(gsi_handle_t h, int* device_status);

gsi_status_t gsi_destroy(gsi_handle_t h);

/* ------------------------------------------------------------------------ *
 * Stack driver: one decode step = every group of every layer, in order, on
 * one stream (Section 1: the method is applied to all linear maps of all
 * layers).  Groups keep their own handles; the stack only chains them.
 *
 * Contract on inputs and order: the inputs x of ALL groups for a step are in
 * device memory before the step is enqueued (gsi_stack_bind).  Groups start in
 * the given order and each group's own chain (projection, residual, gate,
 * image, gated residual) is Algorithm 1, but consecutive groups overlap: a
 * group's gate may be settled, and its W r added, while later groups already
 * project their inputs (the persistent kernel reads a group's x two phases
 * ahead, projects it one phase ahead and settles a gate one phase later;
 * batched stacks run the gated residual contraction of a group beside the
 * kernels of the groups after it).
 * Every y, gate byte and rho of a step is final when the step's work has
 * completed in the order of `stream`, not earlier.
 * ------------------------------------------------------------------------ */

typedef struct {
  const float* x; /* [n_steps][max_tokens][d]: input of this group at every step */
  float* y;       /* [max_tokens][sum d_out]: overwritten at every step          */
} gsi_stack_io_t;

/* Bytes of extra device workspace the stack itself needs (step counter,
 * barrier words, per-group parameter table). */
size_t gsi_stack_workspace_bytes(int n_groups);

/* groups_host_array: HOST array of n_groups handles in execution order; all
 * must have the same max_tokens.  The handles must outlive the stack.  A handle
 * may appear only once in a stack (GSI_ERR_INVALID_ARG otherwise: its scratch and
 * exchange state serve one use per step).  It may belong to several stacks, but
 * only the stack bound LAST may be stepped: gsi_stack_bind resets the handles'
 * cross-CTA exchange state. */
gsi_status_t gsi_stack_create(int n_groups, const gsi_handle_t* groups_host_array,
                              void* workspace, size_t workspace_bytes,
                              gsi_stream_t stream, gsi_stack_t* out);

/*
 * Bind the I/O of every group.  io_host_array: HOST array [n_groups].  The
 * stack keeps a DEVICE-side step counter s; step number s reads
 * x + (s mod n_steps)*max_tokens*d of each group and writes
 *   gate_log[(s mod n_steps)][group][token]   (bytes, may not be NULL)
 *   rho_log [(s mod n_steps)][group][token]   (fp32, may be NULL)
 * so that replaying one captured CUDA graph walks through the pre-staged
 * inputs without host involvement.
 */
gsi_status_t gsi_stack_bind(gsi_stack_t s, const gsi_stack_io_t* io_host_array,
                            int n_steps, unsigned char* gate_log, float* rho_log,
                            gsi_stream_t stream);

/*
 * Declares that groups first_group and first_group + 1 do not read each other's
 * outputs (two branches of one block: in GPT-J the attention output projection
 * and the MLP down projection), so the persistent kernel may run their
 * projections, gates and images at the same time on two parts of the grid
 * (Algorithm 1 itself is unchanged; a gated residual still streams W with the
 * whole grid).  Outside persistent mode (per-stage and batched kernels) the
 * second group of a pair is enqueued on a stream of the stack's own, forked
 * from and joined to the caller's stream by events, so the two chains of
 * launches run side by side (and a stream capture records a fork and a join).
 * Off by default; a group belongs to at most one pair; in persistent mode a
 * pair whose rows do not fit its share of the grid runs one group after the
 * other.  Takes effect at the next gsi_stack_bind.
 */
gsi_status_t gsi_stack_set_concurrent(gsi_stack_t s, int first_group, int enable);

/*
 * Execution mode, taken at the next gsi_stack_bind:
 *   0 (default)  the persistent kernel, one launch per token of the step, when
 *                every group qualifies (one or two tokens per step, no dense
 *                group in a two-token stack, bf16 basis with k in
 *                {64,128,256,512}, d a multiple of 16, rows that fit the
 *                per-CTA buffers), else the per-stage / batched kernels;
 *   1            always the per-stage kernels;
 *   2            the persistent launch or GSI_ERR_UNSUPPORTED from bind.
 * Both modes compute the same layer; they differ in reduction order only.
 */
gsi_status_t gsi_stack_set_mode(gsi_stack_t s, int mode);

/*
 * Polls a cross-CTA wait of the persistent kernel (the exchange of a phase, the
 * arrival counters) may take before it gives up, records GSI_ERR_TIMEOUT in the
 * status word and lets every CTA drain its copies in flight and return; 0
 * restores the default (2^22, about a second).  Waits inside a CTA (its own
 * copies in flight) keep their own, larger limit.  Applies from the next step.
 * A very small value makes the time-out path testable without hanging anything.
 */
gsi_status_t gsi_stack_set_spin_limit(gsi_stack_t s, unsigned polls);

/* 1 if the bound stack runs as one persistent launch per step. */
gsi_status_t gsi_stack_is_persistent(gsi_stack_t s, int* out);

/*
 * Tracing.  `cycles` is a DEVICE array [n_CTAs][GSI_TRACE_SECTIONS] of 64-bit
 * counters (n_CTAs = SM count; NULL switches tracing off).  While set, thread 0
 * of every CTA of the persistent launch adds the SM cycles it spends in each
 * section of the per-phase pipeline:
 *   0 barrier that opens the tick
 *   3 (thread 0 belongs to the warps that wait for the sums; pass 1 and the send of the next
 *     phase run on other warps meanwhile) the statistics hand-over of the phase after the next
 *   4 wait for the sums of the tick's phase, gate of the previous phase, barrier
 *   5 residual rows (with the wait for the basis slab's second copy)
 *   7 image rows (with the waits for the chunks of the image slab)      8 end of the row passes
 *   9 before a W stream                  10 the stream's share of its input into registers
 *  11 wait for W pieces   12 arithmetic on W pieces   13 partial sums into y
 *   6 after the streams of a tick (the grid barrier that follows a dense group)
 * The caller clears and reads the counters.  Applies from the next step.
 */
#define GSI_TRACE_SECTIONS 16
gsi_status_t gsi_stack_set_trace(gsi_stack_t s, unsigned long long* cycles);

/* Set the device-side step counter (enqueued on `stream`). */
gsi_status_t gsi_stack_seek(gsi_stack_t s, int step, gsi_stream_t stream);

/* Enqueue one decode step and advance the device-side counter.  No host
 * synchronisation; may be stream-captured into a CUDA graph and replayed. */
gsi_status_t gsi_stack_step(gsi_stack_t s, gsi_stream_t stream);

/* Number of kernels one gsi_stack_step enqueues (for launch accounting). */
gsi_status_t gsi_stack_launches_per_step(gsi_stack_t s, int* n_out);

/*
 * One decode step with HOST buffers: x_host_array[g] -> device slot of the
 * current step, run the step, copy every group's y and the step's gate bytes
 * back, synchronise.  x_host_array / y_host_array: HOST arrays [n_groups] of
 * HOST pointers ([max_tokens][d] and [max_tokens][sum d_out]); pinned memory
 * makes the copies asynchronous.  gate_host [n_groups][max_tokens].  Groups whose
 * host buffers AND device buffers are adjacent in memory (carved out of one arena, in
 * group order) are copied with a single transfer per direction.
 */
gsi_status_t gsi_stack_step_host(gsi_stack_t s, const float* const* x_host_array,
                                 float* const* y_host_array, unsigned char* gate_host,
                                 gsi_stream_t stream);

/*
 * Synchronises the stack's last stream and returns the device status word (GSI_OK,
 * or GSI_ERR_TIMEOUT if a bounded device-side wait gave up).  After a time-out the
 * outputs of that step are undefined and the cross-CTA exchange state of the
 * persistent kernel is stale: bind the stack again (gsi_stack_bind clears it)
 * before stepping further.
 */
gsi_status_t gsi_stack_get_status(gsi_stack_t s, int* device_status);
gsi_status_t gsi_stack_destroy(gsi_stack_t s);

#ifdef __cplusplus
}
#endif
#endif /* GSI_H_ */
