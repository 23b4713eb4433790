/*
 * mlpmoe.h - C ABI of the B200 (sm_100a) MLPMoE forward library.
 *
 * The layer (arXiv 2511.21089, Section 3.1):
 *     MLPMoE(x) = sum_b alpha_b * W_down^(b) [ silu(W_gate^(b) x) (.) W_up^(b) x ]
 * over B contiguous slices of the intermediate dimension, with Fractal Fade
 * (Section 3.2) and Compensated Branch Pruning (Section 3.3) applied to the
 * weights / gates before the forward pass.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory of the current device, owned by the
 *     caller unless stated otherwise; "host" pointers are ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Every call returns a status; nothing throws or aborts across this boundary.
 *     On error no state of the handle changes.
 *   - One handle may be used from one stream at a time.
 *   - There is no CPU fallback: without a usable CUDA device every compute call
 *     returns MLPMOE_ERR_CUDA.
 *   - Inputs are assumed finite (skipping zeroed work is exact only then).
 */
#ifndef MLPMOE_H_
#define MLPMOE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mlpmoe_layer_s* mlpmoe_handle_t;

typedef enum {
  MLPMOE_OK = 0,
  MLPMOE_ERR_INVALID_ARG = 1,     /* NULL pointer, negative size, n_tokens > max_tokens, misaligned buffer */
  MLPMOE_ERR_BAD_PARTITION = 2,   /* sum d_b != d_inter, d_b <= 0, or d_b not a multiple of 16 */
  MLPMOE_ERR_EMPTY_KEEP_SET = 3,  /* pruning would leave no branch */
  MLPMOE_ERR_BAD_SCHEDULE = 4,    /* a sparsity ratio outside [0, 1) */
  MLPMOE_ERR_UNSUPPORTED = 5,     /* shape or dtype combination the kernels do not cover */
  MLPMOE_ERR_ALLOC = 6,           /* device or host allocation failed */
  MLPMOE_ERR_CUDA = 7,            /* a CUDA runtime / driver call failed (includes: no device) */
  MLPMOE_ERR_DEVICE_TIMEOUT = 8   /* a bounded wait inside a kernel ran out (see mlpmoe_get_status) */
} mlpmoe_status_t;

typedef enum { MLPMOE_BF16 = 0, MLPMOE_FP32 = 1 } mlpmoe_dtype_t;

typedef enum {
  MLPMOE_LAYOUT_PAPER = 0,  /* W_gate, W_up: [d_model x d_inter]; W_down: [d_inter x d_model]; row-major (Section 3.1) */
  MLPMOE_LAYOUT_LINEAR = 1  /* [out x in] row-major: gate/up [d_inter x d_model], down [d_model x d_inter] */
} mlpmoe_layout_t;

/* ------------------------------------------------------------------------- *
 * Set-up calls (may synchronise the stream; allocate library-owned memory)
 * ------------------------------------------------------------------------- */

/*
 * Build a layer from dense SwiGLU weights (Section 3.1: partition of d_inter into
 * B contiguous slices d_inter = sum_b d_b, sub-matrices by slicing, one scalar
 * gate alpha_b per branch).
 *   out        host: receives the handle (NULL on error).
 *   d_b        host, length B: slice widths; each must be a positive multiple of 16.
 *   W_gate, W_up, W_down   device, `dtype` elements in `layout`; copied and packed
 *              on `stream`; the caller may free them once that stream work is done.
 *   alpha      host, length B, or NULL for all 1.0 (the paper's initial value).
 *   dtype      MLPMOE_BF16: bf16 weights and activations, fp32 accumulation on the
 *              tensor cores; MLPMOE_FP32: fp32 everywhere (plain FMA arithmetic).
 *   max_tokens largest n_tokens a later forward call may pass (sizes the
 *              library-owned intermediate-activation workspace).
 * d_model must be a multiple of 8.
 */
mlpmoe_status_t mlpmoe_create(mlpmoe_handle_t* out, int64_t d_model, int64_t d_inter,
                              int32_t B, const int64_t* d_b,
                              const void* W_gate, const void* W_up, const void* W_down,
                              const float* alpha, mlpmoe_dtype_t dtype, mlpmoe_layout_t layout,
                              int64_t max_tokens, void* stream);

/* Free everything the handle owns.  NULL is allowed. */
void mlpmoe_destroy(mlpmoe_handle_t h);

/*
 * Let `h` use `donor`'s intermediate-activation workspace instead of its own (a
 * stack of layers that run one after another on one stream needs only one).
 * `donor` must have been created with at least h's d_inter and max_tokens and
 * the same dtype, and must outlive `h`.  Not in the paper: memory management only.
 */
mlpmoe_status_t mlpmoe_share_workspace(mlpmoe_handle_t h, mlpmoe_handle_t donor);

/*
 * Fractal Fade (Section 3.2, and the "Differential Sparsity Logic" fragment of
 * Section 4): for every branch b with s_b > 0, and separately for its W_gate and
 * its W_up slice (m = d_model * d_b entries each), zero every entry whose
 * magnitude is not above the slice's s_b-quantile of magnitudes.  The quantile
 * position is p = s_b (m - 1) in exact arithmetic; with lo = floor(p) the entries
 * zeroed are exactly those with |w| <= (lo-th smallest |w|), ties included, which
 * is the same set the linearly interpolated threshold with a strict '>' gives.
 * W_down is not touched.  Applied in place to the library's copy; idempotent.
 *   s   host, length B, each in [0, 1); 0 = leave the branch untouched.
 *       NULL = the paper's schedule s_b = 0.9 b / B (b = 0 is the dense backbone),
 *       evaluated in integer arithmetic as lo = (9 b (m - 1)) div (10 B).
 * Afterwards neurons whose gate column, up column or down row is entirely zero are
 * dropped from the schedule.  Synchronises `stream`.
 */
mlpmoe_status_t mlpmoe_fade(mlpmoe_handle_t h, const double* s, void* stream);

/*
 * Neuron-structured Fade: a LABELLED VARIANT of Fractal Fade, not the paper's definition (Section 3.2
 * masks single weights, which saves no work on dense tensor-core tiles; Section 6.2 and Section 7
 * name exactly that gap).  Same schedule, coarser grain: in every branch b with s_b > 0 the
 * q_b = floor(s_b d_b) neurons with the smallest score are removed whole (their W_gate and W_up
 * columns are zeroed; W_down is not touched), where
 *     score_j = sum_k W_gate[k, j]^2 + sum_k W_up[k, j]^2
 * is accumulated in float64 one term after the other in that order (products and sums rounded
 * separately), and ties go to the lower neuron index first.  The removed neurons leave the schedule,
 * so prefill and decode work shrink with them.  s as in mlpmoe_fade (NULL = s_b = 0.9 b / B, with
 * q_b = (9 b d_b) div (10 B)).  Idempotent.  Allocates and frees temporary device memory;
 * synchronises `stream`.
 */
mlpmoe_status_t mlpmoe_fade_structured(mlpmoe_handle_t h, const double* s, void* stream);

/*
 * Compensated Branch Pruning (Section 3.3) with an arbitrary keep set:
 * alpha_b <- alpha_b(create) * sqrt(B / K) for kept branches (K = number kept;
 * factor 1 if `compensate` is 0) and 0 for the others, computed as
 * (float)(sqrt((double)B / K) * (double)alpha_b).  Always starts from the alpha
 * given at create, so repeated calls do not accumulate.  Dropped branches are
 * removed from the packed operands: their work is skipped, not masked.
 *   keep  host, length B, non-zero = keep.  An empty keep set is an error.
 * Synchronises `stream`.
 */
mlpmoe_status_t mlpmoe_prune(mlpmoe_handle_t h, const uint8_t* keep, int32_t compensate, void* stream);

/* The paper's literal rule (Section 3.3): keep branches b < K, alpha_b = sqrt(B/K). 1 <= K <= B. */
mlpmoe_status_t mlpmoe_prune_first_k(mlpmoe_handle_t h, int32_t K, void* stream);

/*
 * Fast fp32 mode for an MLPMOE_FP32 layer: the layer equation of Section 3.1 on the tensor cores at
 * fp32-grade accuracy.  Every fp32 operand v is held as three bf16 pieces p0 = bf16(v),
 * p1 = bf16(v - p0), p2 = bf16(v - p0 - p1) (24 significand bits together); a product a * b is the sum
 * of the six piece products a0 b0, a0 b1, a0 b2, a1 b0, a1 b1, a2 b0 (what is dropped is below
 * 2^-23 of |a b|), accumulated in fp32.  Both GEMMs run this way (the K loop is six times as
 * long), the intermediate activation is kept as the three-way split of its fp32 value, SiLU uses
 * the accurate exponential.  Used by the forward calls for n_tokens > 64; fewer tokens keep the
 * plain fp32 arithmetic.  Enabling allocates the split copies (1.5 x the fp32 weights, and
 * activations for max_tokens) and is re-applied by later fade / prune calls; `enable` = 0 switches
 * back.  MLPMOE_ERR_UNSUPPORTED for a bf16 layer.  Not in the paper: an implementation mode.
 */
mlpmoe_status_t mlpmoe_set_fast_fp32(mlpmoe_handle_t h, int32_t enable, void* stream);

/* ------------------------------------------------------------------------- *
 * Forward (Section 3.1 layer equation).  Enqueues on `stream`, never
 * synchronises, allocates nothing.  (The first call above 128 tokens with a new
 * token count builds that count's tile sequences on the host and uploads them
 * with one asynchronous copy into memory sized at create.)
 * ------------------------------------------------------------------------- */

/*
 *   x  device, [n_tokens x d_model] row-major, the layer's dtype, 16-byte aligned.
 *   y  device, [n_tokens x d_model] row-major, fp32, 16-byte aligned.
 * n_tokens = 0 is a no-op; n_tokens > max_tokens is MLPMOE_ERR_INVALID_ARG.
 * bf16 layers use the tensor-core GEMM pair for n_tokens > 64 and the
 * weight-streaming decode kernels for n_tokens <= 64.
 */
mlpmoe_status_t mlpmoe_forward(mlpmoe_handle_t h, const void* x, void* y, int64_t n_tokens, void* stream);

/*
 * As mlpmoe_forward, with
 *   residual  device fp32 [n_tokens x d_model] or NULL: y = residual + MLPMoE(x)
 *             (may alias y when y_dtype is fp32);
 *   y_dtype   MLPMOE_FP32, or MLPMOE_BF16 for a bf16 layer.
 */
mlpmoe_status_t mlpmoe_forward_ex(mlpmoe_handle_t h, const void* x, void* y, int64_t n_tokens,
                                  const float* residual, mlpmoe_dtype_t y_dtype, void* stream);

/*
 * Per-token branch selection (dynamic routing over branches).  A LABELLED
 * EXTENSION: Section 7 (Limitation 2) and the outlook of Section 8 name routing
 * over the branches as future work and define no rule; the rule here is this
 * library's own, built from Section 3.1's branches and Section 3.3's compensation:
 *     S_t = { b : select[t, b] != 0 and alpha_b != 0 }          (alpha_b: the layer's current gates)
 *     y_t = c_t * sum_{b in S_t} branch_b(x_t),   c_t = sqrt(B' / |S_t|),
 * B' = number of branches with alpha_b != 0; |S_t| = 0 gives y_t = 0; compensate = 0
 * gives c_t = 1.  With every available branch selected this is mlpmoe_forward; with
 * one set shared by all tokens on an unpruned layer it is the layer after
 * mlpmoe_prune(keep = that set).  How the selection is made (a router) is the
 * caller's business.
 *   x       device, [n_tokens x d_model], the layer's dtype, 16-byte aligned
 *   y       device, [n_tokens x d_model] fp32, 16-byte aligned
 *   select  device, [n_tokens x B] row-major bytes
 * Only the selected (token, branch) pairs are computed: the tokens of a branch are
 * gathered into a block of rows of their own, every branch runs on its block as a
 * packed single-branch layer (bf16 layers: all branches in one launch of the
 * persistent CTA-pair kernel; fp32 layers: one mlpmoe_forward per branch), the
 * branch outputs stay fp32 and are summed back per token in ascending b.  The
 * first call, and the first after a Fade or a prune, builds the single-branch
 * layers (allocates about the layer's packed weights once more, plus input,
 * intermediate and fp32 output rows for max_tokens x min(B, 8) selected pairs, and
 * synchronises); EVERY call synchronises `stream` once, to read the per-branch
 * token counts.  Pays for prefill-sized batches; for a handful of tokens the
 * per-branch launches cost more than the skipped branches save.
 * Errors: MLPMOE_ERR_INVALID_ARG (NULL, misaligned, n_tokens > max_tokens),
 * MLPMOE_ERR_ALLOC, MLPMOE_ERR_CUDA.
 */
mlpmoe_status_t mlpmoe_forward_routed(mlpmoe_handle_t h, const void* x, float* y, int64_t n_tokens,
                                      const uint8_t* select, int32_t compensate, void* stream);

/*
 * mlpmoe_forward on HOST buffers: copies x to the device, runs the layer, copies y
 * back and synchronises `stream`.  x_host: layer dtype, y_host: fp32.  Pinned host
 * memory makes the copies asynchronous; pageable memory works too.
 */
mlpmoe_status_t mlpmoe_forward_host(mlpmoe_handle_t h, const void* x_host, float* y_host,
                                    int64_t n_tokens, void* stream);

/* ------------------------------------------------------------------------- *
 * Stack harness (not in the paper; the benchmark configurations wrap the layer
 * as x <- x + MLPMoE_l(RMSNorm(x)), unit gain)
 * ------------------------------------------------------------------------- */

/* r[t,:] = x[t,:] / sqrt(mean(x[t,:]^2) + eps); x device fp32 [n x d]; r device [n x d] of out_dtype. */
mlpmoe_status_t mlpmoe_rmsnorm(const float* x, void* r, int64_t n_tokens, int64_t d_model, float eps,
                               mlpmoe_dtype_t out_dtype, void* stream);

/*
 * Set-up of mlpmoe_stack_forward for this stack (these handles, in this order) and this token
 * count, so that the forward call itself only enqueues: chooses the kernel family, builds the work
 * sequences on the host, allocates the device memory that holds them (and, for up to 128 tokens, a
 * stage-tiled copy of each layer's packed weights, as large as the packed weights; if that memory
 * cannot be had, a slower kernel without the copy), uploads them on `stream` and may synchronise
 * `stream`.  The result is cached in the first layer's handle, one set-up at a time: preparing
 * another token count or stack replaces it, and create / fade / prune on any layer invalidates it.
 * Not in the paper: memory management only.  MLPMOE_ERR_ALLOC if the work sequences cannot be
 * stored (above 128 tokens).
 */
mlpmoe_status_t mlpmoe_stack_prepare(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n_tokens, void* stream);

/*
 * Run n_layers layers (all with the same d_model and dtype) over the fp32 residual
 * stream x [n_tokens x d_model], in place: for each layer, RMSNorm into a
 * library-owned buffer of the layer dtype, then x = x + MLPMoE_l(that).
 *
 * bf16 stacks whose layers share one workspace (mlpmoe_share_workspace) run in one
 * persistent kernel: up to 128 tokens always, above 128 tokens when every layer's
 * packed weights are small enough to stay in L2; other stacks run layer by layer.
 * After mlpmoe_stack_prepare for the same stack and token count the call only
 * enqueues: no allocation, no synchronisation.  Without it (or after a create / fade /
 * prune, or with another token count) the call falls back to doing that set-up itself
 * first, with everything mlpmoe_stack_prepare's comment says about allocation and
 * synchronisation.  Work items add into x in arrival order, so the last bits of the
 * result can differ from run to run.  x: device, 16-byte aligned.
 */
mlpmoe_status_t mlpmoe_stack_forward(const mlpmoe_handle_t* layers, int32_t n_layers, float* x,
                                     int64_t n_tokens, float eps, void* stream);

/* mlpmoe_stack_forward on HOST buffers (fp32 in, fp32 out); synchronises `stream`. */
mlpmoe_status_t mlpmoe_stack_forward_host(const mlpmoe_handle_t* layers, int32_t n_layers,
                                          const float* x_host, float* y_host,
                                          int64_t n_tokens, float eps, void* stream);

/* ------------------------------------------------------------------------- *
 * Queries (host outputs; used by the parity harness)
 * ------------------------------------------------------------------------- */

/*
 * The schedule: surviving branches in ascending order and the maximal runs of
 * live neurons inside them (start index in 0..d_inter-1, length); their
 * concatenation is the contraction index space of the down projection.
 * branches: capacity B; seg_start / seg_len: capacity d_inter.  Any output may be NULL.
 */
mlpmoe_status_t mlpmoe_get_klist(mlpmoe_handle_t h, int32_t* branches, int32_t* n_branches,
                                 int64_t* seg_start, int64_t* seg_len, int32_t* n_segs);
/* Effective alpha_b (after pruning / compensation), length B. */
mlpmoe_status_t mlpmoe_get_alpha(mlpmoe_handle_t h, float* alpha);
/* Number of surviving (scheduled) intermediate neurons. */
mlpmoe_status_t mlpmoe_get_active_neurons(mlpmoe_handle_t h, int64_t* n_active);
/* Non-zero entries per branch of each projection (length B each; any may be NULL). Synchronises. */
mlpmoe_status_t mlpmoe_nnz(mlpmoe_handle_t h, int64_t* nnz_gate, int64_t* nnz_up, int64_t* nnz_down);
/*
 * Copy the library's current weights back in the paper's layout (W_gate, W_up:
 * [d_model x d_inter], W_down: [d_inter x d_model], layer dtype, device buffers;
 * any may be NULL).  After mlpmoe_fade these hold the masked weights.
 */
mlpmoe_status_t mlpmoe_get_weights(mlpmoe_handle_t h, void* W_gate, void* W_up, void* W_down, void* stream);
/*
 * Reads the handle's device status word (synchronises the device): MLPMOE_OK, or
 * MLPMOE_ERR_DEVICE_TIMEOUT if a bounded wait in a kernel ran out since the last call (for a
 * stack call the word of the first layer's handle is the one that is set).  The outputs of
 * the call that timed out, and of every later call on the handle, are undefined until this
 * function has reported the timeout: reporting it also re-arms the handle (clears the word and
 * the dependency counters that a kernel which gave up may have left non-zero), after which
 * the handle can be used again.
 */
mlpmoe_status_t mlpmoe_get_status(mlpmoe_handle_t h);
/*
 * SM clock during the handle's last launch of a persistent kernel (the fused prefill kernel, the
 * prefill-stack kernel, the decode-stack kernels; for a stack call ask the first layer's handle):
 * one thread of the kernel reads the SM cycle counter and the nanosecond wall clock at entry and at
 * exit; sm_mhz = cycles / nanoseconds * 1000, kernel_us = that thread's lifetime.  0 if no such kernel
 * has run.  Synchronises the device.  For benchmarks (not in the paper).
 */
mlpmoe_status_t mlpmoe_get_kernel_clock(mlpmoe_handle_t h, double* sm_mhz, double* kernel_us);
/* Kernels launched on behalf of this handle since create (forward calls only). */
mlpmoe_status_t mlpmoe_get_launch_count(mlpmoe_handle_t h, int64_t* launches);
const char* mlpmoe_status_string(mlpmoe_status_t s);

/*
 * Per-kernel device timing for benchmarks (not in the paper).  With timing enabled, forward
 * calls on this handle record CUDA events on their stream around each kernel they launch;
 * nothing else changes.  Enabling allocates a fixed pool of events (a set-up call); once the
 * pool is used up further launches are simply not timed.
 *   mlpmoe_get_timing synchronises the device and returns, since the last call, the summed
 *   duration in milliseconds and the number of timed launches of: [0] the gate|up kernel,
 *   [1] the down kernel, [2] RMSNorm (stack calls only).  Both arrays have length 3.
 */
mlpmoe_status_t mlpmoe_set_timing(mlpmoe_handle_t h, int32_t enable);
mlpmoe_status_t mlpmoe_get_timing(mlpmoe_handle_t h, double* ms, int64_t* launches);

/* ------------------------------------------------------------------------- *
 * Hooks for tests (not in the paper)
 * ------------------------------------------------------------------------- */

/*
 * Bounded-wait limits of the kernels launched for this handle (for a stack call: the first
 * layer's handle).  limit_ns: how long a wait inside a kernel may last before the kernel gives
 * up, sets the status word and returns (0 = the default of one second).  extra_arrivals is added
 * to the number of arrivals that every wait of one CTA for the work of other CTAs expects; any
 * value above 0 therefore makes those waits run out, which is how the tests reach the give-up
 * path without a fault.  (0, 0) restores normal operation.
 */
mlpmoe_status_t mlpmoe_debug_set_wait(mlpmoe_handle_t h, uint64_t limit_ns, uint32_t extra_arrivals);

/*
 * Which persistent kernel a decode stack call (at most 128 tokens) that starts with this layer runs:
 * 0 = by the library's rule (token count and how many SMs own a neuron tile), 1 = the few-token kernel
 * (both GEMMs on the tile's owner; at most 16 tokens, more tokens fall back to the rule's other kernel),
 * 2 = the kernel with a grid-wide H exchange.  Both compute the same stack; the tests use this to run
 * each of them on shapes where the rule would pick the other.  MLPMOE_ERR_INVALID_ARG for another value.
 */
mlpmoe_status_t mlpmoe_debug_set_decode_kernel(mlpmoe_handle_t h, int32_t kernel);

/*
 * The handle's (possibly shared) activation workspace, for guard-band checks and memory
 * accounting: device addresses and sizes in bytes of H (n x n_active_pad of the layer dtype for
 * an n-token call), of the normalised / staged input (n x d_model, layer dtype) and of the fp32
 * staging buffer of the host-buffer calls (n x d_model), and the current padded neuron count.
 * Any output may be NULL.  The memory stays owned by the library.
 */
mlpmoe_status_t mlpmoe_get_workspace(mlpmoe_handle_t h, void** H, int64_t* H_bytes, void** xnorm, int64_t* xnorm_bytes,
                                     float** yres, int64_t* yres_bytes, int64_t* n_active_pad);

/* ------------------------------------------------------------------------- *
 * Allocation-free variant (the paper has no counterpart: this is a deployment aid)
 * ------------------------------------------------------------------------- */

#define MLPMOE_STATIC_FADE_MAX_SLICES 256

/*
 * The masking step of mlpmoe_fade applied directly to caller-owned device buffers, without a
 * layer handle and without allocating anything: for each slice i (m[i] contiguous elements of
 * `dtype` at slices[i]) every entry with |w| <= (lo-th smallest |w|), lo = floor(s[i] (m[i] - 1))
 * in exact arithmetic, is zeroed in place; s[i] = 0 leaves the slice untouched.  Pass one slice
 * per (branch, projection) to reproduce mlpmoe_fade.
 *
 * For callers that cannot call cudaMalloc when they need this - a process whose device memory
 * was handed to its own arena at start-up, or a path that must avoid cudaMalloc's device-wide
 * synchronisation.  The scratch the selection needs (about 1.1 KB per slice) lives in a fixed
 * array of about 275 KB inside the library image, present on every device that loads the
 * library for the life of the process.  The call uses no cudaMalloc, cudaFree or other
 * allocating routine.
 *   slices, m, s   host arrays of length n_slices (slices holds device pointers, each aligned
 *                  to the element size of `dtype`, else MLPMOE_ERR_INVALID_ARG).
 *   n_slices       at most MLPMOE_STATIC_FADE_MAX_SLICES, else MLPMOE_ERR_UNSUPPORTED.
 * The first call on each device looks up the array's device address (the device must be
 * current).  All calls share the one array: each call re-initialises the part it uses, but two
 * calls whose kernels overlap on the GPU (different streams, or different host threads) race on
 * it - serialise them.  Every call synchronises `stream` before it returns (its segment records
 * are copied from host memory of the call), so it cannot be part of a stream capture.
 */
mlpmoe_status_t mlpmoe_fade_buffers_static(void* const* slices, const int64_t* m, const double* s,
                                           int32_t n_slices, mlpmoe_dtype_t dtype, void* stream);

/* ------------------------------------------------------------------------- *
 * Host-only helpers: the scheduler's integer logic without any CUDA call
 * ------------------------------------------------------------------------- */

/* lo = floor(s (m - 1)) in exact arithmetic on the double s (Section 3.2 quantile position). */
mlpmoe_status_t mlpmoe_host_fade_position(double s, int64_t m, int64_t* lo);
/* lo for the paper's schedule s_b = 0.9 b / B: (9 b (m - 1)) div (10 B). */
mlpmoe_status_t mlpmoe_host_fade_position_default(int32_t b, int32_t B, int64_t m, int64_t* lo);
/* Effective gates of Section 3.3 from create-time alpha and a keep mask. */
mlpmoe_status_t mlpmoe_host_prune_alpha(int32_t B, const float* alpha, const uint8_t* keep,
                                        int32_t compensate, float* alpha_eff);
/*
 * Build the schedule from effective gates and per-neuron liveness flags
 * (live: host uint8[d_inter] or NULL = all live).  Outputs as mlpmoe_get_klist.
 */
mlpmoe_status_t mlpmoe_host_schedule(int32_t B, const int64_t* d_b, const float* alpha_eff,
                                     const uint8_t* live, int32_t* branches, int32_t* n_branches,
                                     int64_t* seg_start, int64_t* seg_len, int32_t* n_segs,
                                     int64_t* n_active);

/*
 * The static tile schedule of the fused prefill kernel for n_tokens tokens: which CTA pair runs
 * which gate|up / down tiles in which order (set-up logic, no CUDA call).  Down tiles are cut into
 * ksplit (1..4) slices of the contraction range.  tiles: capacity
 * ceil(n/256) * (n_active_pad/128 + ksplit * ceil(d_model/bn)); offsets: capacity num_sms/2 + 1.
 * Tile code: bit 31 = down tile, bits 16..30 = column-tile index (down: column tile * ksplit +
 * slice), bits 0..15 = 256-token block.
 */
mlpmoe_status_t mlpmoe_host_tile_schedule(int64_t n_tokens, int64_t d_model, int64_t n_active_pad, int32_t bn,
                                          int32_t ksplit, int32_t num_sms, int32_t* tiles, int32_t* n_tiles,
                                          int32_t* offsets);

/*
 * The work sequences of the persistent prefill-stack kernel (mlpmoe_stack_forward with more than
 * 128 tokens): which CTA pair runs which items of which layer in which order (set-up logic, no
 * CUDA call).  Every pair has two independent sequences: its GEMM items (per layer and 256-token
 * block n_active_pad[l]/128 gate|up tiles and ksplit[l] * ceil(d_model/bn) down items) and the norm
 * parts (16 per layer and block, 16 token rows each) that its norm warps run.  items:
 * item_capacity pairs of int32 (code, layer), code = type << 30 | column << 16 | token block with
 * type 0 = gate|up tile, 1 = down item (column = column tile * ksplit + slice), 2 = norm part
 * (column = part); the GEMM sequences of all pairs come first, then the norm sequences.  *n_items
 * receives the number of items (also when item_capacity is too small, which returns
 * MLPMOE_ERR_INVALID_ARG); offsets: capacity 2 * (num_sms/2 + 1), in items: num_sms/2 + 1 bounds
 * of the GEMM sequences, then num_sms/2 + 1 bounds of the norm sequences.
 */
mlpmoe_status_t mlpmoe_host_stack_schedule(int64_t n_tokens, int64_t d_model, int32_t n_layers, const int64_t* n_active_pad,
                                           const int32_t* ksplit, int32_t bn, int32_t num_sms, int32_t* items,
                                           int64_t item_capacity, int64_t* n_items, int32_t* offsets);

/*
 * The work sequences of the one grouped launch of mlpmoe_forward_routed on a bf16 layer (set-up logic, no
 * CUDA call): block r of the gathered token rows (256 rows) belongs to branch block_branch[r] and has that
 * branch's n_active_pad[b]/128 gate|up tiles and ceil(d_model/bn) down items, nothing else.  items, n_items and
 * the GEMM half of offsets as in mlpmoe_host_stack_schedule, the second int32 of an item being the branch
 * and the token-block field the block index r; the norm sequences (second half of offsets) are empty.
 */
mlpmoe_status_t mlpmoe_host_group_schedule(const int32_t* block_branch, int32_t n_blocks, int64_t d_model, int32_t n_branches,
                                           const int64_t* n_active_pad, int32_t bn, int32_t num_sms, int32_t* items,
                                           int64_t item_capacity, int64_t* n_items, int32_t* offsets);

#ifdef __cplusplus
}
#endif
#endif /* MLPMOE_H_ */
