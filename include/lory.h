/*
 * lory.h -- C ABI of the Lory MoE layer for NVIDIA B200 (sm_100a).
 *
 * The layer is the one defined by "causal segment routing" plus "expert merging"
 * (Section 3.1, Eq. 2, Eq. 3 and Algorithm 1 of the Lory paper):
 *
 *   a sequence of L tokens is cut into N = L/T segments of T tokens;
 *   p_s  = softmax_e( W_r . mean_t x_{s,t} )                         (Eq. 3)
 *   w_s  = p_{s-1} for the 2nd..Nth segment of a sequence, and
 *   w_s  = stop_gradient(p_s) for the first segment                  (Algorithm 1)
 *   theta_bar_s = sum_e w_{s,e} theta_e   for W1, W2, W3             (Eq. 2)
 *   y_t  = W2bar_s ( silu(W1bar_s x_t) * (W3bar_s x_t) )  for every token t of segment s
 *
 * and its backward pass (chain rule through the above; the stop-gradient removes the path
 * from the first segment's weights to W_r and x).
 *
 * Conventions
 *   - Every tensor is dense, row-major, and lives in DEVICE memory unless the argument is
 *     documented as a host pointer.  The caller owns all buffers; this library never
 *     allocates or frees device memory.
 *   - dtype selects the storage type of x, w_r, w1, w2, w3, y, dy, dx, dw_r, dw1, dw2, dw3:
 *     LORY_FP32 (float, fp32 arithmetic throughout) or LORY_BF16 (bfloat16 storage, fp32
 *     accumulation, tensor cores).  route_w, route_p and d_route_w are always float.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream).  Argument errors are detected on the host before anything is launched
 *     and are reported through the return value (a lory_status); nothing throws.
 *   - Gradients are overwritten, not accumulated.
 *   - There is no CPU implementation behind these calls: without a CUDA device of compute
 *     capability 10.x they return LORY_ERR_ARCH / LORY_ERR_CUDA.
 */
#ifndef LORY_H_
#define LORY_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LORY_OK = 0,
  LORY_ERR_NULL = -1,           /* a required pointer is NULL                                  */
  LORY_ERR_SHAPE = -2,          /* a dimension is < 1, L % T != 0, or a size limit is exceeded */
  LORY_ERR_DTYPE = -3,          /* dtype is neither LORY_FP32 nor LORY_BF16                    */
  LORY_ERR_WORKSPACE = -4,      /* workspace smaller than lory_moe_workspace_bytes() says      */
  LORY_ERR_ARCH = -5,           /* current device is not compute capability 10.x               */
  LORY_ERR_CUDA = -6,           /* a CUDA runtime/driver call failed (see lory_last_cuda_error)*/
  LORY_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait expired (lory_check_status)      */
  LORY_ERR_TOO_LARGE = -8,      /* problem exceeds the fixed scratch of lory_route_noalloc     */
  LORY_ERR_DEBUG_BOUNDS = -9    /* debug build: a tile coordinate, shared-memory stage or TMEM
                                   column range was out of bounds (lory_check_status)          */
} lory_status;

typedef enum { LORY_FP32 = 0, LORY_BF16 = 1 } lory_dtype;

/* flags */
#define LORY_FLAG_SIMT 1 /* bf16 only: run every contraction on the plain FMA kernels (diagnostic) */
#define LORY_FLAG_REUSE_MERGED 2 /* lory_moe_ffn only: use the merged weights already in the workspace */
#define LORY_FLAG_PREFIX_ROUTING 4 /* "prefix routing" ablation (Section 5.1): every segment of a sequence is
                                     routed by the sequence's FIRST segment; gradient reaches the router from
                                     segments 2..N only (the first segment's own use keeps the stop-gradient).
                                     Give the same flag to the forward and to the backward call. */
#define LORY_FLAG_FIRST_SEGMENT_GRAD 8 /* backward only: no stop-gradient on the first segment of a sequence, its
                                          own routing weights send gradient to the router (dp_{b,0} += dw_{b,0}).
                                          With T = L (one segment per sequence) this trains the whole-sequence
                                          routing of Section 2.2; the forward is the same with or without it. */
#define LORY_FLAG_ACCUMULATE_GRADS 16 /* backward only: dw_r, dw1, dw2, dw3 receive old value + gradient instead of
                                         the gradient (micro-batches of one optimiser step; the sum is formed in
                                         fp32 and rounded to the storage type).  dx and d_route_w are per call. */

#define LORY_FLAG_CHUNKED_ADJOINT 32 /* backward only, tensor-core pipeline: the per-segment weight gradients (the
                                        adjoint of Eq. 2 needs them for every segment) are formed one rectangle of
                                        one expert matrix at a time in a buffer sized to half the device's L2 and
                                        consumed from there, instead of being written out for the whole matrices.
                                        Same results up to the summation order of the routing gradient; the
                                        backward workspace shrinks by almost the size of the merged weights (2.1 GB
                                        at E = 32, T = 256, d = 1024, f = 2752); two launches per rectangle (68
                                        instead of 4 there) and a slower step (3.5 against 2.7 ms), because this
                                        GPU's L2 writes the buffer back to memory all the same.  Ignored by the
                                        plain-FMA pipeline.  Pass it to lory_moe_workspace_bytes as well; the
                                        buffer size follows the environment variable LORY_ADJOINT_CHUNK_MB (MiB)
                                        when set, read by both calls. */

/*
 * Problem description.  B sequences of L tokens, segment length T (L % T == 0),
 * hidden size d, FFN hidden size f, E experts.
 * In LORY_BF16 mode d and f must be multiples of 8 (16-byte rows for the TMA engine)
 * and E <= 128; with E <= 64 the layer runs on the tensor cores (any B, L, T), with more
 * experts on the slower plain-FMA pipeline.  LORY_FP32 always uses the plain-FMA pipeline.
 */
typedef struct {
  int B, L, T, d, f, E;
  int dtype; /* lory_dtype */
  int flags;
} lory_dims;

/* Human-readable name of a lory_status value.  Never NULL. */
const char* lory_status_string(int status);

/* Text of the last CUDA error this library observed on the calling thread ("" if none). */
const char* lory_last_cuda_error(void);

/*
 * Size in bytes of the scratch buffer the two calls below need.
 *   *fwd_bytes : enough for lory_moe_forward alone;
 *   *bwd_bytes : enough for lory_moe_forward followed by lory_moe_backward (>= *fwd_bytes).
 * Either output pointer may be NULL.  Host-only; launches nothing.
 */
int lory_moe_workspace_bytes(const lory_dims* dims, size_t* fwd_bytes, size_t* bwd_bytes);

/*
 * Forward pass (Algorithm 1 with moe_ffn as in Eq. 2).
 *   x        [B, L, d]    in   layer input
 *   w_r      [E, d]       in   router (bias-free linear layer)
 *   w1, w3   [E, f, d]    in   gate / up projections of the E experts (y = W2 (silu(W1 x) * W3 x))
 *   w2       [E, d, f]    in   down projections
 *   y        [B, L, d]    out
 *   route_w  [B*L/T, E]   out  float, routing weights used by each segment (after the shift)
 *   route_p  [B*L/T, E]   out  float, softmax output of each segment before the shift; may be NULL
 *   workspace             scratch, 256-byte aligned, >= fwd_bytes (>= bwd_bytes if a backward
 *                         call will follow: the forward leaves the merged weights and the FFN
 *                         activations there for it)
 */
int lory_moe_forward(const lory_dims* dims, const void* x, const void* w_r, const void* w1,
                     const void* w2, const void* w3, void* y, float* route_w, float* route_p,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward pass.  Must follow a lory_moe_forward call with the same dims, inputs and
 * workspace on the same stream; the workspace must not be touched in between.
 *   dy         [B, L, d]   in   gradient wrt y
 *   dx         [B, L, d]   out  gradient wrt x, router path included
 *   dw_r       [E, d]      out
 *   dw1, dw3   [E, f, d]   out  dW_e = sum_s w_{s,e} dWbar_s
 *   dw2        [E, d, f]   out
 *   d_route_w  [B*L/T, E]  out  float, <dtheta_bar_s, theta_e>: gradient wrt route_w, the first
 *                               segment's row included although the stop-gradient discards it;
 *                               may be NULL
 */
int lory_moe_backward(const lory_dims* dims, const void* x, const void* w_r, const void* w1,
                      const void* w2, const void* w3, const void* dy, void* dx, void* dw_r,
                      void* dw1, void* dw2, void* dw3, float* d_route_w, void* workspace,
                      size_t workspace_bytes, void* cuda_stream);

/*
 * moe_ffn(seg_x, e) of Algorithm 1 with the routing weights supplied by the caller
 * instead of the router: merge with `route_w` and run the merged SwiGLU FFNs.
 *   x        [S, T, d] (S = B*L/T segments; dims->B, L, T describe the same tokens)
 *   route_w  [S, E]    in, float
 * Uses the same workspace layout as lory_moe_forward (>= fwd_bytes).
 *
 * Inference with prompt-only routing (Section 3.1, "Prompt-only routing during inference"): call
 * lory_moe_forward on the prompt with T = L (one segment per sequence: its routing weights are
 * softmax(R(mean of the prompt)) and its merged FFN processes the prompt); then, for every later
 * chunk of n new tokens per sequence, call lory_moe_ffn with L = T = n and
 * flags | LORY_FLAG_REUSE_MERGED on the SAME workspace: the merge is skipped and the cached merged FFN
 * of each sequence is applied like a dense FFN (route_w is ignored and may be NULL).  B, d, f, E,
 * dtype and LORY_FLAG_SIMT must equal those of the call that merged.
 */
int lory_moe_ffn(const lory_dims* dims, const void* x, const float* route_w, const void* w1,
                 const void* w2, const void* w3, void* y, void* workspace,
                 size_t workspace_bytes, void* cuda_stream);

/*
 * Expert utilisation (appendix "Expert Utilization"): counts[e] = number of the S segments whose
 * routing weight for expert e is larger than 2/E.  route_w [S, E] float and counts [E] int, both DEVICE.
 */
int lory_expert_utilization(const float* route_w, int S, int E, int* counts, void* cuda_stream);

/*
 * The layer inside a pre-norm residual block (Section 4.1: the models follow LLaMA, whose feed-forward sub-layer
 * is y = x + FFN(RMSNorm(x)); the paper does not write the normalisation out, the usual definition is taken):
 *     x_hat = x / sqrt(mean_j x_j^2 + eps) * gamma          per token, fp32 arithmetic, stored in the dtype
 *     y     = x + Lory(x_hat)                               lory_moe_forward on x_hat, then the residual
 * and its backward: gradients of the layer as in lory_moe_backward (taken at x_hat), then
 *     dx     = RMSNorm backward of dL/dx_hat  +  dy         (the residual path)
 *     dgamma = sum over tokens of dL/dx_hat * x * inv_rms
 * The workspace keeps x_hat and the per-token inverse rms from the forward for the backward, in front of the
 * layer's own workspace.
 *   x, dy, y, dx   [B, L, d] DEVICE          gamma, dgamma [d] DEVICE (same dtype)       eps >= 0
 *   every other argument as in lory_moe_forward / lory_moe_backward; flags apply to the layer inside
 *   (LORY_FLAG_ACCUMULATE_GRADS also accumulates dgamma).
 *   workspace      DEVICE scratch of >= lory_block_workspace_bytes() bytes, 256-byte aligned
 * Errors: as the layer calls; LORY_ERR_SHAPE for a negative or NaN eps.
 */
int lory_block_workspace_bytes(const lory_dims* dims, size_t* forward_bytes, size_t* backward_bytes);
int lory_block_forward(const lory_dims* dims, const void* x, const void* gamma, float eps, const void* w_r,
                       const void* w1, const void* w2, const void* w3, void* y, float* route_w,
                       float* route_p, void* workspace, size_t workspace_bytes, void* cuda_stream);
int lory_block_backward(const lory_dims* dims, const void* x, const void* gamma, const void* w_r,
                        const void* w1, const void* w2, const void* w3, const void* dy, void* dx,
                        void* dgamma, void* dw_r, void* dw1, void* dw2, void* dw3, float* d_route_w,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * One training step of the layer driven from HOST activations: copies x and dy from
 * host memory to the device, runs forward and backward, and copies y, dx and route_w back.
 * The parameters and their gradients stay on the device (they are optimiser state, not
 * per-step input).  dY travels to the device while the forward runs and y travels back while the
 * backward runs (an internal second stream, created on first use).  Synchronises the stream
 * before returning.
 *   x_host, dy_host       [B, L, d]  in   HOST (pinned for full copy speed)
 *   y_host, dx_host       [B, L, d]  out  HOST
 *   route_w_host          [S, E]     out  HOST float
 *   w_r, w1, w2, w3, dw_r, dw1, dw2, dw3   DEVICE, as in the two calls above
 *   arena                 DEVICE scratch of >= lory_moe_step_host_bytes() bytes, 256-byte aligned
 */
int lory_moe_step_host_bytes(const lory_dims* dims, size_t* arena_bytes);
int lory_moe_step_host(const lory_dims* dims, const void* x_host, const void* dy_host,
                       const void* w_r, const void* w1, const void* w2, const void* w3,
                       void* y_host, void* dx_host, float* route_w_host, void* dw_r, void* dw1,
                       void* dw2, void* dw3, void* arena, size_t arena_bytes, void* cuda_stream);

/*
 * The same step as a two-slot pipeline, for a training loop that feeds one batch after another from host
 * memory: lory_moe_step_host_enqueue() only enqueues (copy in, forward, backward, copy out) and returns;
 * lory_moe_step_host_wait() blocks until the outputs of the step last enqueued on that slot are in host
 * memory.  With the slots used alternately (step i on slot i & 1), the host-to-device copy of step i+1 and
 * the device-to-host copy of step i-1 run while step i computes (three streams: an internal copy-in stream,
 * the caller's stream for the kernels, an internal copy-out stream, ordered by events).  Results are those
 * of lory_moe_step_host.  Rules: host buffers of a slot must stay untouched between its enqueue and its
 * wait; each slot needs its own y_host, dx_host and route_w_host; wait on a slot before enqueuing on it
 * again; one pipeline per host thread.  Parameter gradients (dw_r, dw1, dw2, dw3) are overwritten by every
 * step, in stream order.
 *   slot                  0 or 1
 *   arena                 DEVICE scratch of >= lory_moe_step_host_pipeline_bytes() bytes, 256-byte aligned,
 *                         shared by both slots
 * Errors: as lory_moe_step_host; LORY_ERR_SHAPE for a slot other than 0 or 1.
 */
int lory_moe_step_host_pipeline_bytes(const lory_dims* dims, size_t* arena_bytes);
int lory_moe_step_host_enqueue(const lory_dims* dims, int slot, const void* x_host, const void* dy_host,
                               const void* w_r, const void* w1, const void* w2, const void* w3,
                               void* y_host, void* dx_host, float* route_w_host, void* dw_r, void* dw1,
                               void* dw2, void* dw3, void* arena, size_t arena_bytes, void* cuda_stream);
int lory_moe_step_host_wait(int slot);

/*
 * Reads the device status word kept in the workspace (synchronises the stream).
 * Returns LORY_OK, or LORY_ERR_DEBUG_BOUNDS if a bounds check of the debug build fired, or
 * LORY_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up; in both cases the outputs of that
 * call are undefined.
 */
int lory_check_status(const lory_dims* dims, void* workspace, size_t workspace_bytes,
                      void* cuda_stream);

/*
 * Routing step without any caller-supplied or freshly allocated scratch.  (The paper has no
 * counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a plug-in inside a
 * serving process whose memory was handed out in full at start-up, a control loop that must not hit
 * cudaMalloc because that call may stall every stream of the device, or a host that passes this
 * library nothing but input and output pointers and has no allocator to size a workspace with.
 *
 * It computes what the first stage of lory_moe_forward computes: segment means, router softmax and
 * the causal shift (Eq. 3, Algorithm 1), i.e. route_w and route_p, from x and w_r.  The intermediate
 * segment means and probabilities go to a fixed array of LORY_NOALLOC_SCRATCH_BYTES that is part of
 * the library image; every GPU that loads the library holds that array until the process exits.
 * The call performs no cudaMalloc/cudaFree and calls nothing that allocates.
 *
 *   x        [B, L, d]   in   DEVICE, dims->dtype
 *   w_r      [E, d]      in   DEVICE, dims->dtype
 *   route_w  [B*L/T, E]  out  DEVICE float, weights after the shift
 *   route_p  [B*L/T, E]  out  DEVICE float, softmax before the shift; may be NULL
 *   dims->f is ignored.
 *
 * Limit: (S*d + S*E) * 4 bytes, S = B*L/T, must not exceed LORY_NOALLOC_SCRATCH_BYTES; larger
 * problems return LORY_ERR_TOO_LARGE and launch nothing.
 * Every call looks up the array's device address (cudaGetSymbolAddress) for the current device and keeps no
 * copy of it, so a context that was reset in between is harmless.  The first call on a device also loads the
 * library's device code there: make that first call outside any stream capture.
 * All calls on one device share the one array, and it keeps the previous call's contents.  Nothing in
 * it needs clearing (every element is rewritten before it is read), but two calls whose kernels can
 * overlap on the GPU -- different streams, or different host threads -- race on it: keep calls on one
 * device ordered on a single stream.
 */
#define LORY_NOALLOC_SCRATCH_BYTES (4u << 20)
int lory_route_noalloc(const lory_dims* dims, const void* x, const void* w_r, float* route_w,
                       float* route_p, void* cuda_stream);

/*
 * Self-test of the failure path: launches a one-thread kernel that waits, with a small poll limit, on a
 * barrier nothing ever completes.  The wait must give up and raise the workspace's status word, so that a
 * following lory_check_status returns LORY_ERR_DEVICE_TIMEOUT (and the device stays usable).  Clears the
 * status word first.  The kernels of the layer use the same bounded wait with a much larger limit.
 */
int lory_selftest_bounded_wait(const lory_dims* dims, void* workspace, size_t workspace_bytes,
                               void* cuda_stream);

/*
 * Debug build.  The library can be built a second time with -DLORY_DEBUG
 * (python -m paper_2405_03133_b200.build --debug -> liblory_debug.so; same ABI).  Its tensor-core kernels
 * check, before use, every tile coordinate they hand to the TMA engine (range against the padded problem
 * extents, 16-byte alignment of the innermost coordinate), every shared-memory stage and staging buffer
 * against the CTA's allocation, and every TMEM column range against the allocated columns.  A violated
 * bound sets a bit in the status word and the access is skipped (stores, MMAs) or redirected to coordinate
 * zero (loads) rather than issued; lory_check_status then returns LORY_ERR_DEBUG_BOUNDS.  This is the
 * tool for hunting an out-of-range index without a memory checker; it costs a few per cent of run time.
 *   lory_debug_build()            1 in the debug build, 0 in the release build.
 *   lory_selftest_debug_bounds()  makes the three kinds of check fire on purpose, on made-up values and
 *                                 without any access: in the debug build a following lory_check_status
 *                                 returns LORY_ERR_DEBUG_BOUNDS, in the release build LORY_OK (the checks
 *                                 are compiled out).  Clears the status word first.
 */
int lory_debug_build(void);
int lory_selftest_debug_bounds(const lory_dims* dims, void* workspace, size_t workspace_bytes,
                               void* cuda_stream);

/*
 * Optional per-launch timing.  lory_profile_enable(1) clears the record list and makes every
 * later call bracket each of its kernels (or kernel groups) with two CUDA events on the call's
 * stream; lory_profile_enable(0) stops recording.  lory_profile_read waits for the recorded
 * events and writes up to max_records (label, milliseconds) pairs in launch order; it returns
 * the number written (>= 0) or a negative lory_status.  Labels are static strings owned by the
 * library.  At most 8192 records are kept.  Not thread-safe; meant for benchmarks.
 */
int lory_profile_enable(int on);
int lory_profile_read(int max_records, const char** labels, float* ms);

/*
 * Diagnostic (the paper has no counterpart): bandwidth of a write-then-read-back ring in device memory, the
 * measurement behind the decision where the per-segment merged weights and their gradients travel between the
 * kernel that writes them and the kernel that reads them (HBM or the L2 cache).
 * The ring has `slots` regions of `slot_bytes` (rounded down to a whole number of 16-byte vectors per thread).
 * Twice as many CTAs as the device has SMs each own one slice of every slot; in iteration i a CTA writes its
 * slice of slot i mod slots (mode bit 0) and reads the slice of the CTA `shift` positions further in slot
 * (i - lag) mod slots (mode bit 1), with loads and stores that bypass L1.  Reads hit L2 while
 * (lag + 1) * slot_bytes still fits there.  One untimed pass fills the ring, then `iters` iterations are timed
 * with CUDA events; the call synchronises the stream.  Bytes moved: iters * slot_bytes per active direction.
 *   buf      DEVICE scratch, 256-byte aligned, >= slots * slot_bytes + 256 bytes
 *   ms_out   HOST float, duration of the timed pass in milliseconds
 * Errors: LORY_ERR_NULL, LORY_ERR_SHAPE (slots < 1, lag outside [0, slots], iters < 1, mode outside 1..3,
 * shift < 0, slot too small), LORY_ERR_WORKSPACE (buffer too small or misaligned), LORY_ERR_CUDA.
 */
int lory_probe_l2_ring(void* buf, size_t buf_bytes, size_t slot_bytes, int slots, int lag, int iters, int mode,
                       int shift, float* ms_out, void* cuda_stream);

/* Number of kernel launches issued by the last forward / backward call on this thread. */
int lory_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LORY_H_ */
