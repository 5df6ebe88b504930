/*
 * mixlora.h - C ABI of the MixLoRA feed-forward block for NVIDIA B200 (sm_100a).
 *
 * The block is the one defined by Eq. 6-9 and Algorithm 1 of "MixLoRA: Enhancing Large
 * Language Models Fine-Tuning with LoRA-based Mixture of Experts" (arXiv 2404.15159):
 * a frozen SwiGLU FFN (W1 = gate, W3 = up, W2 = down; Section 3.3) shared by N LoRA
 * experts (Eq. 1: W' = W + B A on each of the three projections) under a top-k softmax
 * router (Eq. 7) with the load-balance auxiliary loss of Eq. 8-9.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer unless marked "host".  All tensors are
 *     dense, row-major, 16-byte aligned and owned by the caller, including the workspace.
 *     The library allocates no device memory in these calls.  What a call computes depends only on its
 *     arguments and the workspace; the process-wide state the library keeps is scheduling plumbing: a few streams
 *     and events per device that calls borrow between a fork and a join (see mixlora_ffn_forward), a table of
 *     encoded tensor maps, the switches of mixlora_set_option and the opt-in bookkeeping of mixlora_stage_timing.
 *     Calls may be made from several host threads (different workspaces).
 *   - Weights are stored [out, in] as in Eq. 1 (W in R^{d1 x d2}).
 *   - T tokens, d = d_model, f = d_ff, N experts, k = top_k, r = rank, s = lora_alpha / r.
 *     A slot is one (token, selected expert) pair; slot id = t * k + j, j = 0 for the
 *     expert with the largest logit.
 *   - dtype 0: x, dy, y, d_x, frozen weights and LoRA matrices are bfloat16, arithmetic
 *     accumulates in fp32.  dtype 1: all of them are fp32 (check mode).  Router weight,
 *     router bias, probabilities, gates and every gradient output are fp32 in both modes.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*); calls return after
 *     enqueueing and never synchronise the device (mixlora_device_status excepted).
 *   - Errors: every call validates its arguments on the host and returns a status; nothing
 *     aborts or throws.  A failed validation enqueues nothing.
 */
#ifndef MIXLORA_H_
#define MIXLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MIXLORA_OK = 0,
  MIXLORA_ERR_INVALID_ARG = 1,   /* NULL or misaligned pointer, inconsistent sizes            */
  MIXLORA_ERR_UNSUPPORTED = 2,   /* a size outside the compiled limits (see mixlora_limits)  */
  MIXLORA_ERR_WORKSPACE = 3,     /* workspace NULL, misaligned or smaller than required      */
  MIXLORA_ERR_CUDA = 4,          /* a CUDA runtime or driver call failed                     */
  MIXLORA_ERR_DEVICE_TIMEOUT = 5 /* a bounded wait inside a kernel ran out (device status)   */
} mixlora_status_t;

#define MIXLORA_DTYPE_BF16 0
#define MIXLORA_DTYPE_FP32 1

#define MIXLORA_MAX_EXPERTS 32   /* N <= 32                                              */
#define MIXLORA_MAX_TOP_K 8      /* k <= min(N, 8)                                       */
#define MIXLORA_MAX_MODELS 16    /* adapters per multi-model call                         */
#define MIXLORA_MAX_RANK 128     /* r <= 128; r % 8 == 0 in bf16 mode, r % 4 == 0 in fp32 */

/* Problem shape.  Plain data; set struct_size = sizeof(mixlora_shape_t). */
typedef struct {
  uint32_t struct_size;
  int32_t tokens;       /* T >= 0 (T = 0 is a valid no-op); T * k <= 4,000,000                */
  int32_t d_model;      /* d, multiple of 8                                                  */
  int32_t d_ff;         /* f, multiple of 8                                                  */
  int32_t n_experts;    /* N                                                                 */
  int32_t top_k;        /* k, 1 <= k <= N                                                    */
  int32_t rank;         /* r                                                                 */
  float lora_alpha;     /* scale s = lora_alpha / rank (alpha of Table 3)                    */
  int32_t dtype;        /* MIXLORA_DTYPE_BF16 or MIXLORA_DTYPE_FP32                          */
  int32_t renormalize;  /* 1: gates divided by their top-k sum (Norm(.) of Algorithm 1); 0: Eq. 7 as printed */
  int32_t aux_f_mode;   /* 0: F_i counts the arg-max expert (Eq. 9); 1: all k selections / (T k)            */
} mixlora_shape_t;

/* Inputs of the block.  `void*` tensors have the element type selected by shape.dtype. */
typedef struct {
  const void *x;               /* [T, d]  hidden states (after the layer norm of Eq. 5)      */
  const void *w_gate;          /* [f, d]  W1, frozen                                         */
  const void *w_up;            /* [f, d]  W3, frozen                                         */
  const void *w_down;          /* [d, f]  W2, frozen                                         */
  const float *w_router;       /* [N, d]  W_r of Eq. 7, fp32                                 */
  const float *router_bias;    /* [N] fp32 added to the logits, or NULL                      */
  const void *a_gate, *b_gate; /* [N, r, d], [N, f, r]                                       */
  const void *a_up, *b_up;     /* [N, r, d], [N, f, r]                                       */
  const void *a_down, *b_down; /* [N, r, f], [N, d, r]                                       */
} mixlora_params_t;

/* Gradient outputs, fp32 (d_x in shape.dtype), same shapes as the parameter they belong to.
 * A NULL pointer skips that gradient.  The frozen weights never get one. */
typedef struct {
  float *d_a_gate, *d_b_gate;
  float *d_a_up, *d_b_up;
  float *d_a_down, *d_b_down;
  float *d_w_router;          /* [N, d] */
  float *d_router_bias;       /* [N]    */
  void *d_x;                  /* [T, d] or NULL                                               */
  int32_t accumulate;         /* 0: overwrite the fp32 outputs; 1: add to them (gradient
                                 accumulation, Table 3).  d_x is always overwritten.          */
} mixlora_grads_t;

/* Compiled limits, for callers that size things ahead of time. */
typedef struct {
  int32_t max_experts, max_top_k, max_rank;
} mixlora_limits_t;
void mixlora_limits(mixlora_limits_t *out /* host */);

/* Bytes of workspace that forward (for_backward = 0) or forward followed by backward
 * (for_backward = 1) need for this shape.  Returns 0 if the shape is invalid. */
size_t mixlora_workspace_bytes(const mixlora_shape_t *shape /* host */, int for_backward);

/* Forward pass: y = sum_j g_tj * E_{e_tj}(x_t)  (Eq. 6 through Algorithm 1).
 * Steps, all on the device: router logits, softmax, top-k, gates (Eq. 7); slot histogram,
 * prefix scan and stable permutation by expert; shared W1/W3 projections once per token
 * (Section 3.3 (I)); per-expert LoRA deltas; SwiGLU; down projection plus its LoRA; gate-
 * weighted combine.  `y` is [T, d] in shape.dtype.  The routing, the probabilities and the
 * activations that the backward pass re-uses are left in `workspace` (256-byte aligned).
 * The router and the dispatch are enqueued on a stream that the library creates on first use (one set per device,
 * kept until exit) so that they run beside the shared projections; they start after everything enqueued on
 * `stream` before the call, and the rest of the call, like later work on `stream`, starts after them.
 * mixlora_set_option(MIXLORA_OPT_SERIAL, 1) keeps every launch on `stream`. */
mixlora_status_t mixlora_ffn_forward(const mixlora_shape_t *shape /* host */,
                                     const mixlora_params_t *params /* host struct of device ptrs */,
                                     void *y, void *workspace, size_t workspace_bytes, void *stream);

/* Auxiliary load-balance loss of Eq. 8-9 from the routing that the last forward call left
 * in `workspace`: loss = coef * N * sum_i F_i * P_i.  `loss` is a device scalar; `F`, `P`
 * are device arrays of N floats or NULL. */
mixlora_status_t mixlora_aux_loss(const mixlora_shape_t *shape /* host */, const void *workspace, float coef,
                                  float *loss, float *F, float *P, void *stream);

/* Eq. 8-9 when the batch is spread over data-parallel shards (the paper trains on one GPU; F_i and P_i are
 * fractions of the WHOLE batch, so the loss of the batch is not the mean of the shards' losses, but the sums over
 * tokens that F_i and P_i are built from add up over shards).
 * mixlora_aux_stats copies, from the routing that the last forward call left in `workspace`, the un-normalised sums
 * of this call's tokens into two device arrays of N floats: prob_sum[i] = sum_t p_t[i], count[i] = tokens whose
 * arg-max expert is i (aux_f_mode 1: selections that went to i).  The caller adds both over its shards (one
 * all-reduce of 2N floats) and hands the totals, with the token count of the whole batch, to
 * mixlora_aux_loss_global, which returns loss = coef * N * sum_i F_i P_i of the whole batch (`loss` device scalar,
 * `F`, `P` device [N] or NULL) and leaves F_i and the batch's token count in `workspace`: a backward call that
 * follows then differentiates the batch's loss (d L_aux / d p_t[i] = coef N F_i / total_tokens), so that the shards'
 * gradients add up to the gradient of the whole batch.  Without this call the backward pass uses this call's own
 * tokens, as mixlora_aux_loss does.  total_tokens >= shape->tokens. */
mixlora_status_t mixlora_aux_stats(const mixlora_shape_t *shape /* host */, const void *workspace, float *prob_sum,
                                   float *count, void *stream);
mixlora_status_t mixlora_aux_loss_global(const mixlora_shape_t *shape /* host */, void *workspace, float coef,
                                         const float *prob_sum, const float *count, int64_t total_tokens,
                                         float *loss, float *F, float *P, void *stream);

/* Backward pass of L = <dy, y> + aux_coef * N * sum_i F_i P_i with respect to the LoRA
 * matrices, the router and, if grads->d_x is not NULL, x (chain rule on Algorithm 1; the
 * paper prints no backward).  Needs the workspace exactly as the forward call for the same
 * shape and params left it (size for_backward = 1).  `dy` is [T, d] in shape.dtype.  As in the forward call, a few
 * small launches (the gate-gradient sums, the router's backward step) go to a library-owned stream that forks from
 * and joins `stream` inside the call. */
mixlora_status_t mixlora_ffn_backward(const mixlora_shape_t *shape /* host */,
                                      const mixlora_params_t *params /* host struct of device ptrs */,
                                      const void *dy, float aux_coef, void *workspace, size_t workspace_bytes,
                                      const mixlora_grads_t *grads /* host struct of device ptrs */, void *stream);

/* mixlora_ffn_backward for data-parallel training (the paper trains on one GPU; the block is independent per token
 * except for the sums over tokens in the LoRA / router gradients, so replicas hold their own tokens and sum those
 * gradients).  Same arguments and results; in addition `param_grads_ready` (a cudaEvent_t created by the caller, or
 * NULL) is recorded on `stream` as soon as every LoRA and router gradient has been enqueued, which is before the
 * input-gradient product (the longest launch of the backward pass, and it writes no parameter gradient).  A caller
 * that waits for the event on a second stream and all-reduces the gradients there overlaps the collective with that
 * product. */
mixlora_status_t mixlora_ffn_backward_overlap(const mixlora_shape_t *shape /* host */,
                                              const mixlora_params_t *params /* host struct of device ptrs */,
                                              const void *dy, float aux_coef, void *workspace, size_t workspace_bytes,
                                              const mixlora_grads_t *grads /* host struct of device ptrs */,
                                              void *param_grads_ready /* cudaEvent_t or NULL */, void *stream);

/* Multi-model forward and backward (Section 3.3 (II), the task loop of Algorithm 1): n_models MixLoRA adapters,
 * each with its own tokens, router, experts, rank and workspace, share ONE frozen FFN (same w_gate, w_up, w_down
 * pointers, same d_model, d_ff and dtype; anything else returns MIXLORA_ERR_INVALID_ARG).  The frozen weights are
 * held once, and the adapters' tokens pass through W1 / W3 (forward) and W2 (backward) two adapters per launch;
 * every other step runs per adapter exactly as in the single-model calls, so each adapter's results equal those of
 * mixlora_ffn_forward / mixlora_ffn_backward on it alone, bit for bit.  All arrays are HOST arrays of n_models
 * entries (of structs / device pointers / sizes); workspaces and outputs must be distinct per adapter.
 * mixlora_aux_loss and mixlora_routing_view are called per adapter on its own workspace.
 * The per-adapter steps of different adapters are enqueued on a few streams that the library creates on first use
 * (one set per device, kept until exit); they start after everything enqueued on `stream` before the call, and work
 * enqueued on `stream` after the call starts after them. */
mixlora_status_t mixlora_multi_ffn_forward(int32_t n_models, const mixlora_shape_t *shapes /* host [n] */,
                                           const mixlora_params_t *params /* host [n] */, void *const *y /* host [n] */,
                                           void *const *workspaces /* host [n] */,
                                           const size_t *workspace_bytes /* host [n] */, void *stream);
mixlora_status_t mixlora_multi_ffn_backward(int32_t n_models, const mixlora_shape_t *shapes /* host [n] */,
                                            const mixlora_params_t *params /* host [n] */,
                                            const void *const *dy /* host [n] */, const float *aux_coef /* host [n] */,
                                            void *const *workspaces /* host [n] */,
                                            const size_t *workspace_bytes /* host [n] */,
                                            const mixlora_grads_t *grads /* host [n] */, void *stream);

/* The block inside its transformer layer (Eq. 5 / Eq. 6): h = MixLoRA(LN(z)) + z, with LN the root-mean-square
 * normalisation of LLaMA-class models, xn = norm_weight * z / sqrt(mean(z^2) + eps) over the model width.
 * params->x is z, the residual stream [T, d]; norm_weight is [d]; both, like xn, h, dh and grads->d_x, are device
 * arrays of shape.dtype.  The forward call writes xn [T, d] and inv_rms [T] (fp32), which the caller owns and must
 * pass unchanged to the backward call, together with the workspace as the forward call left it.  The residual is
 * added in the down projection's epilogue; nothing else differs from mixlora_ffn_forward on xn.
 * The backward call returns the LoRA and router gradients of mixlora_ffn_backward at xn and, in grads->d_x (may be
 * NULL), dL/dz = dh + J_LN^T dL/dxn; norm_weight is frozen and gets no gradient.  xn, h and d_x must not alias z or
 * each other; d_model <= 8192 (bf16) or 4096 (fp32), else MIXLORA_ERR_UNSUPPORTED.  mixlora_aux_loss and
 * mixlora_routing_view work on the workspace as after mixlora_ffn_forward. */
mixlora_status_t mixlora_layer_forward(const mixlora_shape_t *shape /* host */,
                                       const mixlora_params_t *params /* host struct of device ptrs */,
                                       const void *norm_weight, float eps, void *xn, float *inv_rms, void *h,
                                       void *workspace, size_t workspace_bytes, void *stream);
mixlora_status_t mixlora_layer_backward(const mixlora_shape_t *shape /* host */,
                                        const mixlora_params_t *params /* host struct of device ptrs */,
                                        const void *norm_weight, float eps, const void *xn, const float *inv_rms,
                                        const void *dh, float aux_coef, void *workspace, size_t workspace_bytes,
                                        const mixlora_grads_t *grads /* host struct of device ptrs */, void *stream);

/* MixDoRA (Section 4.1 and Table 1 name the variant: MixLoRA with every expert's LoRA replaced by DoRA; the paper
 * prints no formula, so this is the weight-decomposed form as it is commonly applied to a linear layer).  Each of
 * an expert's three projections becomes
 *     W'_e = diag(m_e / n_e) (W + s B_e A_e),   n_e[o] = || W[o, :] + s B_e[o, :] A_e ||_2,
 * with one trainable magnitude per output feature and expert (m_gate, m_up [N, f], m_down [N, d], fp32) and the
 * norm n_e, recomputed from the current weights in every forward call, treated as a constant by the backward pass.
 * With m = n the block is MixLoRA; with B = 0 and m = the row norms of W it is the frozen FFN.  Router, gates,
 * dispatch and auxiliary loss are those of mixlora_ffn_forward; W1 x and W3 x are still computed once per token
 * (the scale acts on output rows), while W2 is applied per slot, because the scale of its output differs between
 * a token's experts.  The workspace has its own size (mixlora_dora_workspace_bytes) and layout; mixlora_aux_loss,
 * mixlora_routing_view and mixlora_device_status work on it as after mixlora_ffn_forward.  The backward call needs
 * the workspace as the forward call for the same arguments left it and returns, besides the gradients of
 * mixlora_ffn_backward, those of the magnitudes (fp32, same shapes; NULL skips one; `accumulate` of `grads`
 * applies to them too).  Every step runs on `stream`. */
typedef struct {
  const float *m_gate, *m_up; /* [N, f] */
  const float *m_down;        /* [N, d] */
} mixlora_dora_t;
typedef struct {
  float *d_m_gate, *d_m_up;   /* [N, f] or NULL */
  float *d_m_down;            /* [N, d] or NULL */
} mixlora_dora_grads_t;
size_t mixlora_dora_workspace_bytes(const mixlora_shape_t *shape /* host */, int for_backward);
mixlora_status_t mixlora_dora_ffn_forward(const mixlora_shape_t *shape /* host */,
                                          const mixlora_params_t *params /* host struct of device ptrs */,
                                          const mixlora_dora_t *magnitudes /* host struct of device ptrs */, void *y,
                                          void *workspace, size_t workspace_bytes, void *stream);
mixlora_status_t mixlora_dora_ffn_backward(const mixlora_shape_t *shape /* host */,
                                           const mixlora_params_t *params /* host struct of device ptrs */,
                                           const mixlora_dora_t *magnitudes /* host struct of device ptrs */,
                                           const void *dy, float aux_coef, void *workspace, size_t workspace_bytes,
                                           const mixlora_grads_t *grads /* host struct of device ptrs */,
                                           const mixlora_dora_grads_t *magnitude_grads /* host struct of device ptrs */,
                                           void *stream);

/* Plain LoRA on a linear layer (Eq. 1, W' = W + B A, applied as in Section 3.2 to the attention projections of
 * a MixLoRA model): y = x W^T + s (x A^T) B^T with s = lora_alpha / rank.  x [T, d_in], W [d_out, d_in] (frozen),
 * A [rank, d_in], B [d_out, rank], y and dy [T, d_out], all device arrays of shape.dtype; d_in, d_out and rank are
 * multiples of 8, rank <= MIXLORA_MAX_RANK.  The low-rank term is computed as `rank` extra reduction columns of the
 * frozen product (forward) and of the input-gradient product (backward).  The workspace (256-byte aligned, caller-
 * owned, mixlora_lora_linear_workspace_bytes) keeps s x A^T between the forward and the backward call of the same
 * input.  The backward call writes d_a [rank, d_in] and d_b [d_out, rank] in fp32 (added to the old contents if
 * accumulate = 1) and d_x [T, d_in] in shape.dtype; each may be NULL.  mixlora_lora_linear_status reads back the
 * device status word of the last calls on this workspace (0 = ok; it synchronises the stream). */
typedef struct {
  uint32_t struct_size; /* = sizeof(mixlora_linear_shape_t) */
  int32_t tokens, d_in, d_out, rank;
  float lora_alpha;
  int32_t dtype;        /* MIXLORA_DTYPE_* */
} mixlora_linear_shape_t;
size_t mixlora_lora_linear_workspace_bytes(const mixlora_linear_shape_t *shape /* host */);
mixlora_status_t mixlora_lora_linear_forward(const mixlora_linear_shape_t *shape /* host */, const void *x,
                                             const void *w, const void *a, const void *b, void *y, void *workspace,
                                             size_t workspace_bytes, void *stream);
mixlora_status_t mixlora_lora_linear_backward(const mixlora_linear_shape_t *shape /* host */, const void *x,
                                              const void *w, const void *a, const void *b, const void *dy,
                                              void *workspace, size_t workspace_bytes, float *d_a, float *d_b,
                                              void *d_x, int32_t accumulate, void *stream);
int32_t mixlora_lora_linear_status(const void *workspace, void *stream);

/* Device pointers into the workspace, for inspection after a forward call:
 * expert_idx [T, k] (descending logit), gates [T, k], perm [T*k] (slot id at each position
 * of the order "expert ascending, token ascending"), seg_off [N+1] (first position of each
 * expert), low_margin [T] (1 where a logit gap deciding the top-k set or the arg-max is
 * below 1e-4), probs [T, N].  Any output pointer may be NULL. */
mixlora_status_t mixlora_routing_view(const mixlora_shape_t *shape /* host */, const void *workspace,
                                      const int32_t **expert_idx, const float **gates, const int32_t **perm,
                                      const int32_t **seg_off, const uint8_t **low_margin, const float **probs);

/* Reads the device status word of the workspace (synchronises `stream`).  *code is 0 when
 * no kernel reported a problem, else the mixlora_status_t the kernel recorded. */
mixlora_status_t mixlora_device_status(const void *workspace, int32_t *code /* host */, void *stream);

/* Dense product C[M, N] = A[M, K] * op(B) on the tensor-core path used for the frozen
 * projections (the W1/W3/W2 products of Algorithm 1 and their transposes in the backward
 * pass), exposed so that it can be tested and timed on its own.  A is [M, K] row-major
 * bf16.  b_is_kn = 0: B is [N, K] row-major (a weight stored [out, in]); b_is_kn = 1: B is
 * [K, N] row-major (the same weight used transposed).  C is [M, N] row-major bf16.
 * K and N must be multiples of 8.  `status_word` is a device int32 that receives a non-zero
 * code if a bounded wait in the kernel runs out, or NULL. */
mixlora_status_t mixlora_gemm_bf16(const void *A, const void *B, void *C, int32_t M, int32_t N, int32_t K,
                                   int32_t b_is_kn, int32_t *status_word, void *stream);

/* Slot dispatch without a workspace (the paper has no counterpart; it computes what the
 * dispatch step of mixlora_ffn_forward computes).  For callers that cannot allocate device
 * memory and so have no workspace to pass: a plug-in inside a host program that owns the
 * allocator, code that must not trigger the device-wide synchronisation of cudaMalloc, a
 * process with a memory budget fixed at start-up.  The per-block count tables that the
 * dispatch kernels need between their three launches sit in a 64 KiB array that is part of
 * the library image on every GPU that loads it (held until the process exits).
 *   expert_idx [tokens, top_k] int32 device, values in [0, n_experts), distinct per token.  An entry outside
 *         [0, n_experts) is skipped (it is counted nowhere and leaves one trailing position of perm unwritten); an
 *         expert repeated within a token makes that token's slots share a position.  Neither reads or writes
 *         outside the arrays.
 *   perm  [tokens * top_k] int32 device out: slot id (t * top_k + j) at each position of the
 *         order "expert ascending, token ascending".
 *   seg_off [n_experts + 1] int32 device out: first position of each expert.
 * Limits: tokens <= mixlora_dispatch_static_max_tokens() (65536), n_experts <= 32,
 * top_k <= 8; larger sizes return MIXLORA_ERR_UNSUPPORTED and enqueue nothing.
 * The call allocates nothing, on the device or through any library.  The first call on each
 * device looks up the device address of the array (with that device current); make that
 * first call outside any stream capture.  All calls on a device share the one array: it
 * keeps whatever the last call left, every entry a call reads is written by that call
 * first, and two calls whose kernels overlap on the GPU (different streams, no ordering)
 * race on it - keep such calls ordered. */
mixlora_status_t mixlora_dispatch_static(const int32_t *expert_idx, int32_t tokens, int32_t n_experts,
                                         int32_t top_k, int32_t *perm, int32_t *seg_off, void *stream);
int32_t mixlora_dispatch_static_max_tokens(void);

/* Process-wide switches (they change how work is scheduled, never a result).  value is 0 or 1.
 *   MIXLORA_OPT_SERIAL    1: every launch goes to the caller's stream; the library uses no stream of its own.
 *                         Default 0, or 1 when MIXLORA_SERIAL=1 is in the environment at the first call.
 *   MIXLORA_OPT_TC_SINGLE 1: the dense products use the single-CTA tensor-core kernel for every shape instead of
 *                         CTA pairs (a measurement switch).  Default 0, or 1 with MIXLORA_TC_SINGLE=1. */
#define MIXLORA_OPT_SERIAL 0
#define MIXLORA_OPT_TC_SINGLE 1
mixlora_status_t mixlora_set_option(int32_t option, int32_t value);

/* Failure-path check that faults nothing: launches one thread that waits, for at most `wait_rounds` polls
 * (1 .. 2^20), on a barrier nothing ever signals - the bounded wait every kernel of this library uses - and then
 * records MIXLORA_ERR_DEVICE_TIMEOUT in the status word at the start of `workspace` (256-byte aligned device
 * memory, at least 256 bytes), exactly as a production kernel does when one of its waits runs out.
 * mixlora_device_status then reads 5; the context stays usable. */
mixlora_status_t mixlora_selftest_wait_timeout(void *workspace, uint32_t wait_rounds, void *stream);

/* Opt-in bookkeeping for measurements (host side, process-wide).
 * mixlora_stage_timing(1) clears the counters and makes every later forward / backward /
 * aux_loss call bracket each stage of the path (router, dispatch, the dense products, the
 * LoRA stages, ...) with CUDA events on the caller's stream; mixlora_stage_timing(0) clears
 * and switches the events off (kernel launches are still counted).
 * mixlora_stage_timing_read waits for the recorded events and fills, for up to max_stages
 * stages, the stage name (static string), the device milliseconds accumulated since the last
 * mixlora_stage_timing call and the number of kernels launched.  Returns the number of stages. */
mixlora_status_t mixlora_stage_timing(int32_t enable);
int32_t mixlora_stage_timing_read(int32_t max_stages, const char **names /* host */, float *ms /* host */,
                                  int64_t *launches /* host */);

const char *mixlora_status_string(mixlora_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* MIXLORA_H_ */
