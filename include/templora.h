/*
 * templora.h -- C ABI of the B200 (sm_100a) Temp-Lora chunk-update library.
 *
 * The library runs the per-chunk inference-time update of a temporary LoRA
 * module (Algorithm 1 of the Temp-Lora paper, the training step of the module Theta_k;
 * hyper-parameters of the "Setup" paragraph) for LoRA-augmented linear projections, and
 * the decode-time forward used between updates (Algorithm 1, generation step).
 *
 * Notation (row-major, contiguous rows, no bias):
 *     x  [T, d_in]       chunk activations           W0 [d_out, d_in]  frozen base weight
 *     A  [r, d_in]       LoRA down-projection        B  [d_out, r]     LoRA up-projection
 *     y, dY [T, d_out]   output / upstream gradient  dX [T, d_in]      input gradient
 *     U = x A^T [T, r]   V = dY B [T, r]             s = alpha / r     (paper: 64/64)
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer unless stated otherwise; descriptor
 *     arrays (templora_linear_t[], templora_param_t[], pointer arrays) are HOST arrays.
 *   - The caller owns every buffer, the workspace included.  The library allocates
 *     no device memory, frees nothing, never writes W0, and never synchronises the
 *     stream (templora_read_device_status excepted).  All work is enqueued on
 *     `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - dtype TEMPLORA_BF16: x, W0, A, B, y, dY, dX are bfloat16; products accumulate
 *     in fp32; gradients dA, dB, optimizer moments and master parameters are fp32.
 *     dtype TEMPLORA_F32: everything is fp32.
 *   - Data pointers must be 16-byte aligned.  The tensor-core path (bf16, d_in, d_out
 *     and r multiples of 8, r <= 256) is taken automatically; other shapes run on a
 *     generic kernel path.  r <= 256 always (the paper sweeps rank 16..256).
 *   - Workspace: 256-byte aligned, at least templora_*workspace_bytes() long, and its
 *     first 1024 bytes zeroed by the caller once before first use (they hold the
 *     device status record and the kernels' work counters and flags, which every
 *     kernel leaves at zero; zero them again after a TEMPLORA_ERR_TIMEOUT was
 *     recorded).  A workspace must not be shared by calls that may overlap on the GPU.
 *   - Synchronous errors (bad argument, unsupported shape, short workspace, a CUDA
 *     launch failure) are returned and nothing further is launched.  Device-side
 *     problems (a bounded wait inside a kernel ran out) are recorded in the status
 *     record at the head of the workspace; read it with templora_read_device_status.
 */
#ifndef TEMPLORA_H_
#define TEMPLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TEMPLORA_OK = 0,
  TEMPLORA_ERR_INVALID_ARG = 1,   /* NULL/misaligned pointer, non-positive size          */
  TEMPLORA_ERR_UNSUPPORTED = 2,   /* shape or dtype outside what the kernels handle       */
  TEMPLORA_ERR_WORKSPACE = 3,     /* workspace NULL, misaligned or too small              */
  TEMPLORA_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                    */
  TEMPLORA_ERR_TIMEOUT = 5        /* a bounded device-side wait expired (device status)   */
} templora_status_t;

typedef enum { TEMPLORA_F32 = 0, TEMPLORA_BF16 = 1 } templora_dtype_t;

/* One LoRA-augmented projection (the temporary module attached to one frozen linear). */
typedef struct {
  int32_t d_in, d_out, r;
  float s;            /* alpha / r                                                  */
  int32_t dtype;      /* templora_dtype_t: storage type of x, W0, A, B, y, dY, dX   */
  const void *W0;     /* [d_out, d_in]  frozen, read only                           */
  const void *A;      /* [r, d_in]      working copy in `dtype`                     */
  const void *B;      /* [d_out, r]     working copy in `dtype`                     */
  /* LoRA dropout on the input of the low-rank branch during the update (paper's Setup:
   * dropout = 0.05).  0 disables it.  The keep mask of an [T, d_in] input is drawn from
   * Philox4x32-10: element e = t*d_in + k takes word e % 4 of the block with counter
   * (lo(e/4), hi(e/4), lo(offset), hi(offset)) and key (lo(seed), hi(seed)), and is dropped
   * iff that word < floor(p * 2^32).  templora_linear_fwd and templora_linear_bwd use
   * offset = dropout_offset (pass the same value to both); templora_update_block adds the
   * number of optimizer steps already taken, so every step draws a new mask.  The
   * decode-time forward never drops.  */
  float dropout_p;
  /* Projections that read the same input (q, k, v of one block; gate and up): give them the same
   * nonzero input_group and the same dX buffer in templora_update_block*, and that buffer receives
   * the SUM of their input gradients, i.e. the gradient with respect to the shared input, formed in
   * one accumulator.  At most three projections per group, equal d_in, all within one run of eight
   * consecutive projections starting at a multiple of eight.  0 = on its own (dX, if given, is this
   * projection's own gradient, as in templora_linear_bwd).  Ignored by the other entry points.  */
  int32_t input_group;
  uint64_t dropout_seed;
  uint64_t dropout_offset;
} templora_linear_t;

/* Optimizer state of one tensor (an A or a B); all buffers caller-owned, n elements. */
typedef struct {
  int64_t n;
  float *master;      /* fp32 parameter that AdamW updates                           */
  float *m, *v;       /* fp32 first and second moments                               */
  void *work;         /* copy in the working dtype re-emitted after each step
                         (bf16, round-to-nearest-even); NULL when master is itself
                         what the projections read (fp32 path)                       */
  const float *grad;  /* fp32 gradient (dA or dB)                                    */
} templora_param_t;

/* Bytes of workspace sufficient for templora_linear_fwd, templora_linear_bwd and
 * templora_decode_fwd on this projection with up to T rows.  0 on invalid input. */
size_t templora_workspace_bytes(const templora_linear_t *lin, int32_t T);

/* Bytes of workspace sufficient for templora_update_block on these projections. */
size_t templora_update_block_workspace_bytes(const templora_linear_t *proj, int32_t n_proj, int32_t T);

/*
 * Forward of the LoRA-augmented projection over a chunk of T tokens
 * (module forward inside the training step of Theta_k, Algorithm 1; LoRA of the Section "Temp-Lora"):
 *     U = x A^T ;  y = x W0^T + s U B^T
 * (with dropout_p > 0:  U = xd A^T,  xd = x * keep / (1 - p))
 * x [T,d_in] in, y [T,d_out] out.  U_save: optional fp32 [T,r] that receives U
 * (unscaled) for reuse by templora_linear_bwd; NULL to skip.
 */
templora_status_t templora_linear_fwd(const templora_linear_t *lin, int32_t T, const void *x, void *y,
                                      float *U_save, void *ws, size_t ws_bytes, void *stream);

/*
 * Backward of the same projection with W0 frozen (the method never alters the base
 * model, so there is no dW0):
 *     V = dY B ;  dX = dY W0 + s V A ;  dB = s dY^T U ;  dA = s V^T x
 * (with dropout_p > 0:  dX = dY W0 + s (V A) * keep / (1 - p),  dA = s V^T xd)
 * U_saved: fp32 [T,r] from the forward, or NULL to recompute U = x A^T.
 * dX [T,d_in] may be NULL (skipped).  dA [r,d_in], dB [d_out,r] are fp32 and are
 * plain sums over the T tokens (no 1/T); accumulate != 0 adds to their contents.
 */
templora_status_t templora_linear_bwd(const templora_linear_t *lin, int32_t T, const void *x, const void *dY,
                                      const float *U_saved, void *dX, float *dA, float *dB, int32_t accumulate,
                                      void *ws, size_t ws_bytes, void *stream);

/*
 * One AdamW step (decoupled weight decay, bias-corrected) on n_params tensors
 * (optimizer step of the training step of Theta_k, Algorithm 1; learning rate 5e-5 in the paper's Setup,
 * fp32 master weights and moments as bfloat16 ZeRO-2 training implies):
 *     p <- p (1 - lr wd);  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2
 *     p <- p - lr (m / (1-b1^step)) / (sqrt(v / (1-b2^step)) + eps)
 * `step` is the 1-based index of this step.  params is a HOST array.
 * If work_dtype is TEMPLORA_BF16 and work != NULL, work receives bf16(p).
 */
templora_status_t templora_adamw_step(const templora_param_t *params, int32_t n_params, float lr, float beta1,
                                      float beta2, float eps, float weight_decay, int64_t step,
                                      int32_t work_dtype, void *stream);

/*
 * Decode-time forward with the current (un-merged) module for n_tokens in 1..16 rows
 * (generation step Y[i] = Theta_k(...) of Algorithm 1):  y = x W0^T + s (x A^T) B^T.
 * Streams W0 once per call; bound by HBM bandwidth.  On the tensor-core path the call is one kernel launch
 * whose counters and flags in the workspace head are re-armed on the device, so after one call outside a
 * capture (one-time set-up per device and kernel) it, and templora_decode_block_fwd, may be recorded into a CUDA
 * graph and replayed with new contents in the same x buffer.
 */
templora_status_t templora_decode_fwd(const templora_linear_t *lin, int32_t n_tokens, const void *x, void *y,
                                      void *ws, size_t ws_bytes, void *stream);

/*
 * Decode-time forward of n_proj independent projections in one call (same formula and token
 * limit as templora_decode_fwd).  Projections that do not depend on one another - q, k, v of
 * one block, or gate and up - share launches: every W0 is still streamed exactly once, but
 * the launch and pipeline ramp-up cost is paid once per group of up to 8 projections instead
 * of once per projection.  proj, x, y are HOST arrays; x[i] [n_tokens, d_in_i] and
 * y[i] [n_tokens, d_out_i] are device pointers.
 */
size_t templora_decode_block_workspace_bytes(const templora_linear_t *proj, int32_t n_proj);
templora_status_t templora_decode_block_fwd(const templora_linear_t *proj, int32_t n_proj, int32_t n_tokens,
                                            const void *const *x, void *const *y, void *ws, size_t ws_bytes,
                                            void *stream);

/*
 * The whole chunk update of n_proj projections: for each of `epochs` epochs, forward
 * and backward of every projection over the T-token chunk with the current A, B, then
 * one AdamW step on every A and B (batch = chunk, so one optimizer step per epoch;
 * "n epochs" of Algorithm 1, n = 2 in the paper).
 *   proj[i].A / .B must alias A_state[i].work / B_state[i].work (bf16) or .master (fp32);
 *   gradients are written to A_state[i].grad / B_state[i].grad (cast away const inside:
 *   the buffers are outputs of this call);
 *   x[i] [T,d_in_i], dY[i] [T,d_out_i] inputs, constant across epochs;
 *   y[i] [T,d_out_i] outputs (last epoch); dX[i] [T,d_in_i] outputs, dX or entries may be NULL.
 *   *step_inout: number of optimizer steps already taken; incremented once per epoch.
 * proj, A_state, B_state, x, dY, y, dX, step_inout are HOST memory.
 */
templora_status_t templora_update_block(const templora_linear_t *proj, const templora_param_t *A_state,
                                        const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                        const void *const *x, const void *const *dY, void *const *y,
                                        void *const *dX, int32_t epochs, float lr, float beta1, float beta2,
                                        float eps, float weight_decay, int64_t *step_inout,
                                        void *ws, size_t ws_bytes, void *stream);

/*
 * The same update with the chunk cut into batches of batch_tokens rows (the last may be
 * shorter): forward, backward and one AdamW step per batch, so each epoch takes
 * ceil(T / batch_tokens) optimizer steps (the paper's cost table: chunk 2048, batch 1024,
 * 2 epochs = 4 steps).  batch_tokens >= T is templora_update_block.  Gradient buffers hold
 * the last batch's gradients on return.
 */
templora_status_t templora_update_block_batched(const templora_linear_t *proj, const templora_param_t *A_state,
                                                const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                                int32_t batch_tokens, const void *const *x, const void *const *dY,
                                                void *const *y, void *const *dX, int32_t epochs, float lr,
                                                float beta1, float beta2, float eps, float weight_decay,
                                                int64_t *step_inout, void *ws, size_t ws_bytes, void *stream);

/*
 * Linear learning-rate warm-up ("Setup": the rate is warmed up linearly over the first two
 * chunks).  Rate of optimizer step `step` (1-based, counted over the whole run):
 * lr * min(1, step / warmup_steps); warmup_steps <= 0 gives lr.  For the paper's setting pass
 * warmup_steps = 2 * epochs * ceil(chunk / batch).  Host function, no GPU work.
 */
float templora_lr_at_step(float lr, int64_t step, int64_t warmup_steps);

/*
 * templora_update_block_batched with that warm-up applied inside the call: the optimizer step
 * numbered k = *step_inout + 1, + 2, ... uses templora_lr_at_step(lr, k, warmup_steps).
 * warmup_steps = 0 is templora_update_block_batched.
 */
templora_status_t templora_update_block_warmup(const templora_linear_t *proj, const templora_param_t *A_state,
                                               const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                               int32_t batch_tokens, const void *const *x, const void *const *dY,
                                               void *const *y, void *const *dX, int32_t epochs, float lr,
                                               int64_t warmup_steps, float beta1, float beta2, float eps,
                                               float weight_decay, int64_t *step_inout, void *ws, size_t ws_bytes,
                                               void *stream);

/* Static description of a status code. */
const char *templora_status_string(templora_status_t st);

/*
 * Synchronises `stream`, then copies the device status record at the head of `ws`
 * into *code (a templora_status_t; TEMPLORA_OK if no kernel reported a problem) and
 * *where (an internal location tag).  Returns TEMPLORA_OK if the record was read.
 */
templora_status_t templora_read_device_status(void *ws, void *stream, int32_t *code, int32_t *where);

/*
 * The element-wise steps on either side of the projections when the training step of Theta_k (Algorithm 1) runs over
 * a Llama-style decoder block: the MLP's gating between gate/up and down, and the RMSNorm in front of
 * q,k,v and of gate,up.  The paper names neither (it trains stock Llama-2 / Yi blocks); the formulas are
 * those models' definitions.  All tensors are contiguous DEVICE buffers of `dtype` (templora_dtype_t),
 * 16-byte aligned; arithmetic in fp32; nothing is allocated; errors as for the other entry points.
 *
 * SiLU gating over n elements (any shape, flattened):
 *   fwd:  h = SiLU(gate) * up,            SiLU(g) = g * sigmoid(g)
 *   bwd:  dgate = dh * up * SiLU'(gate),  dup = dh * SiLU(gate),  SiLU'(g) = sigmoid(g) (1 + g (1 - sigmoid(g)))
 */
templora_status_t templora_swiglu_fwd(int64_t n, int32_t dtype, const void *gate, const void *up, void *h, void *stream);
templora_status_t templora_swiglu_bwd(int64_t n, int32_t dtype, const void *gate, const void *up, const void *dh,
                                      void *dgate, void *dup, void *stream);

/*
 * RMSNorm over the rows of x [T, d] with weight w [d] (frozen: no weight gradient):
 *   fwd:  y[t, j]  = x[t, j] * rstd[t] * w[j],   rstd[t] = 1 / sqrt(mean_j x[t, j]^2 + eps)
 *   bwd:  dx[t, j] = rstd[t] * (w[j] dy[t, j] - xh[t, j] * mean_j(xh[t, j] w[j] dy[t, j])),  xh = x * rstd
 * The backward recomputes rstd from x.
 */
templora_status_t templora_rmsnorm_fwd(int32_t T, int32_t d, int32_t dtype, const void *x, const void *w, float eps,
                                       void *y, void *stream);
templora_status_t templora_rmsnorm_bwd(int32_t T, int32_t d, int32_t dtype, const void *x, const void *w, const void *dy,
                                       float eps, void *dx, void *stream);

/*
 * The chunk update of the MLP of a Llama-style decoder block in one call (the training step of Theta_k, Algorithm 1, run over
 * the block's gate, up and down projections with the gating between them; the gating is the model's, see above):
 *     gate = x Wg^T + s (x Ag^T) Bg^T     up = x Wu^T + s (x Au^T) Bu^T     h = SiLU(gate) * up
 *     y    = h Wd^T + s (h Ad^T) Bd^T
 * and, from dY (the gradient with respect to y), the backward through down, the gating and gate/up:
 *     dh = dY Wd + s (dY Bd) Ad;  dgate, dup as in templora_swiglu_bwd;
 *     dX = dgate Wg + dup Wu + s (dgate Bg) Ag + s (dup Bu) Au      (the gradient with respect to x)
 * with the six LoRA gradients as in templora_linear_bwd, then one AdamW step on all six tensors; `epochs` times.
 *   proj, A_state, B_state: HOST arrays of three entries in the order gate, up, down, aliased as in
 *   templora_update_block; gate.d_in == up.d_in, gate.d_out == up.d_out == down.d_in; dropout_p must be 0.
 *   x [T, d_in], dY [T, down.d_out] inputs; gate, up, h [T, d_ff] and y [T, down.d_out] outputs (gate and up are the
 *   pre-activations the backward reads); dX [T, d_in] output or NULL.  All device buffers of the projections' dtype.
 * On the tensor-core path the gating costs no pass of its own: gate and up are one GEMM whose epilogue also
 * writes h, and dh is never stored: the epilogue of the down projection's input gradient writes dgate and dup.
 */
size_t templora_update_mlp_workspace_bytes(const templora_linear_t *proj, int32_t T);
templora_status_t templora_update_mlp(const templora_linear_t *proj, const templora_param_t *A_state,
                                      const templora_param_t *B_state, int32_t T, const void *x, const void *dY,
                                      void *gate, void *up, void *h, void *y, void *dX, int32_t epochs, float lr,
                                      float beta1, float beta2, float eps, float weight_decay, int64_t *step_inout,
                                      void *ws, size_t ws_bytes, void *stream);

/*
 * The chunk update of the projections that read a decoder block's normalised input, in one call (the training
 * step of Theta_k, Algorithm 1, run over RMSNorm -> q, k, v of a Llama-style block; the norm is the model's, its
 * weight frozen):
 *     xn  = RMSNorm(x; norm_weight, norm_eps)                          (as templora_rmsnorm_fwd)
 *     y_i = xn W_i^T + s_i (xn A_i^T) B_i^T                            i = 0 .. n_proj-1, n_proj <= 3
 * and, from the dY_i:
 *     dXn = sum_i (dY_i W_i + s_i (dY_i B_i) A_i)      ONE summed gradient with respect to xn, formed in the
 *                                                      accumulator of one GEMM (as templora_linear_t.input_group)
 *     dX  = RMSNorm backward of dXn                                    (as templora_rmsnorm_bwd)
 * with the LoRA gradients as in templora_linear_bwd and one AdamW step on all A_i, B_i; `epochs` times (x does not
 * change between epochs, so xn is formed once; dXn and dX are the last epoch's).
 *   proj, A_state, B_state: HOST arrays of n_proj entries, aliased as in templora_update_block; equal d_in and dtype
 *   (input_group is ignored: the projections share their input by construction).  dY, y: HOST arrays of n_proj
 *   device pointers.  x [T, d_in], norm_weight [d_in] inputs; xn, dXn [T, d_in] outputs; dX [T, d_in] output or NULL.
 *   Workspace: templora_update_block_workspace_bytes(proj, n_proj, T).
 */
templora_status_t templora_update_attn_in(const templora_linear_t *proj, const templora_param_t *A_state,
                                          const templora_param_t *B_state, int32_t n_proj, int32_t T, const void *x,
                                          const void *norm_weight, float norm_eps, const void *const *dY, void *xn,
                                          void *const *y, void *dXn, void *dX, int32_t epochs, float lr, float beta1,
                                          float beta2, float eps, float weight_decay, int64_t *step_inout, void *ws,
                                          size_t ws_bytes, void *stream);

/*
 * Failure-detection self-test (the paper has no counterpart).  Enqueues one tiny kernel that
 * waits, the way the GEMM kernels wait for their copies, on a barrier that nothing signals.
 * After limit_ms (1..1000) it records TEMPLORA_ERR_TIMEOUT in the status record at the head of
 * `ws` and returns normally: templora_read_device_status then reports the code, and the stream
 * and context stay usable.  Zero the workspace head again afterwards.
 */
templora_status_t templora_selftest_bounded_wait(void *ws, size_t ws_bytes, int32_t limit_ms, void *stream);

/*
 * Parallelized deployment (the paper's "Further Analysis": update the module in a second process or
 * stream while generation continues, then swap it in).  Caps the number of SMs that the
 * library's persistent kernels occupy when launched on `stream`, so that a chunk update on
 * one stream and the decode-time forward on another run side by side instead of taking
 * turns: e.g. 116 SMs for the update stream and 32 for the decode stream on a 148-SM B200.
 * max_sms = 0 removes the cap.  Process-wide table keyed by the stream handle.
 */
templora_status_t templora_set_stream_sm_limit(void *stream, int32_t max_sms);

/*
 * Parallelized deployment with disjoint SMs ("Further Analysis", same passage).  A cap alone bounds how many SMs a
 * stream's kernels ask for, not which ones, so the two sides still get in each other's way at every kernel
 * boundary.  templora_sm_partition_create splits the current device's SMs into two fixed groups and creates one
 * stream in each (driver green contexts): kernels launched on stream_first only ever run on the first group's
 * SMs, those on stream_rest on the others.  first_sms is rounded by the driver to its granularity (8 SMs on
 * sm_100); sms_first / sms_rest report what each side got, and the matching per-stream caps are set.
 *   - `out` is a HOST struct filled by the call; the streams are cudaStream_t handles owned by the partition
 *     (non-blocking with respect to the legacy default stream) and may be used with any CUDA call.
 *   - Device memory, tensor maps and workspaces are shared with the rest of the process as usual.
 *   - TEMPLORA_ERR_UNSUPPORTED when the driver offers no SM partitioning; nothing is created then.
 *   - templora_sm_partition_destroy synchronises both streams, destroys them and releases the groups.
 */
typedef struct {
  void *handle;          /* opaque */
  void *stream_first;    /* cudaStream_t */
  void *stream_rest;     /* cudaStream_t */
  int32_t sms_first, sms_rest;
} templora_sm_partition_t;
templora_status_t templora_sm_partition_create(int32_t first_sms, templora_sm_partition_t *out);
templora_status_t templora_sm_partition_destroy(templora_sm_partition_t *part);

/*
 * Kernel-path selection for testing: 0 = automatic (tensor-core path when the
 * shape allows, frozen-weight GEMMs on CTA pairs), 1 = always the generic kernel path,
 * 2 = tensor-core path with single-CTA tiles only (decode then runs as a W0 stream with
 * split-K partials in the workspace plus a finishing kernel instead of the one-kernel cluster
 * form).  Returns the previous value.
 * Process-wide; not part of the method.
 */
int32_t templora_set_kernel_path(int32_t mode);

/*
 * templora_decode_fwd for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).  Some hosts of this library are handed
 * only input and output buffers and may not call cudaMalloc themselves: a serving loop whose
 * device memory belongs entirely to another framework's pool, a latency-critical thread for
 * which an allocation (which may synchronise the device) is off limits, a plug-in without an
 * allocator.  This variant takes no workspace.  Its scratch is a fixed array of
 * TEMPLORA_NOALLOC_SCRATCH_BYTES inside the library image, present on every GPU that loads
 * the library for the life of the process.  The call allocates and frees nothing.
 *   - Same arguments and result as templora_decode_fwd, minus the workspace.
 *   - A projection whose decode scratch would exceed the array is refused with
 *     TEMPLORA_ERR_UNSUPPORTED and nothing is launched (all Llama-2 7B- and 70B-shaped
 *     projections at rank 64 fit).
 *   - The first call on each device looks up the array's device address; make that first
 *     call with the device current and before starting any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents
 *     (the call clears the part that must start at zero).  Two calls that may overlap on the
 *     GPU, e.g. on different streams, race on it: serialise them, or use templora_decode_fwd
 *     with one workspace per stream.
 *   - Arguments are checked as in templora_decode_fwd before anything is enqueued; a refused
 *     call leaves the array untouched.
 *   - The device status record of this variant lives at the head of the array and is cleared
 *     when an accepted call starts, so it describes the most recent call only.  Read it with
 *     templora_decode_fwd_noalloc_status, which does what templora_read_device_status does
 *     (synchronises `stream`, copies the record out) and allocates nothing either.
 */
#define TEMPLORA_NOALLOC_SCRATCH_BYTES (8u << 20)
templora_status_t templora_decode_fwd_noalloc(const templora_linear_t *lin, int32_t n_tokens, const void *x,
                                              void *y, void *stream);
templora_status_t templora_decode_fwd_noalloc_status(void *stream, int32_t *code, int32_t *where);

/*
 * Launch accounting, a profiling aid (the paper has no counterpart).  The library counts
 * the launches of each kernel class; for the classes selected by kind_mask (bit k = class k,
 * -1 = all, 0 = none) it also records a pair of CUDA events on the launching stream around
 * every launch (which costs the timed kernel and its successor their early scheduling).  Kernel classes: 0 tensor-core GEMM
 * with 256-wide tiles (y, dX), 1 tensor-core GEMM with 64-wide tiles (U, V, dA, dB),
 * 2 tensor-core GEMM with 16-wide tiles (decode), 3 partial reduction, 4 AdamW,
 * 5 generic GEMM, 6 decode finish, 7 dropout mask, 8 masked rank-r pass of dX, 9 SiLU gating and
 * RMSNorm.  Process-wide.
 */
void templora_timing_enable(int32_t kind_mask);

/*
 * Waits for the recorded events of class `kind` and returns their summed device time
 * (*total_ms), how many launches were timed and how many were counted since the last
 * reset.  reset != 0 clears the class afterwards.  Output pointers may be NULL.
 */
templora_status_t templora_timing_read(int32_t kind, double *total_ms, int64_t *timed_launches,
                                       int64_t *all_launches, int32_t reset);

#ifdef __cplusplus
}
#endif
#endif /* TEMPLORA_H_ */
