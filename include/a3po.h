/*
 * a3po.h — C ABI of the B200 (sm_100a) A-3PO log-prob + loss library.
 *
 * The library computes the data-parallel hot path of one A-3PO training step:
 *   hidden states --LM head + log-softmax + gather--> log pi_theta(a_t|s_t)
 *   --> A-3PO decoupled clipped loss with the staleness-interpolated proximal anchor
 *   --> dL/dlogp --> dL/dhidden, dL/dW_lmhead.
 *
 * Conventions for every entry point (unless an argument says otherwise):
 *   - Pointers are DEVICE pointers owned by the caller.  The library allocates no device
 *     memory: scratch space is the caller's `ws` buffer (size it with the *_workspace_bytes
 *     functions; 256-byte aligned).  Contents of `ws` are undefined before and after a call.
 *     Besides that, the library's device image holds two fixed arrays per GPU: 8 KB of
 *     counters with which the CTAs of a tensor-core launch keep in step (advisory, all zero
 *     between launches), and the scratch of a3po_loss_fwd_static.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = legacy default
 *     stream).  Calls never synchronise the device and are asynchronous w.r.t. the host.
 *     A call with device inputs is a fixed sequence of launches (row counts stay on the
 *     device), so it may be captured into a CUDA graph and replayed; make one uncaptured call
 *     per device first (it resolves kernel attributes and the addresses of the library's
 *     device arrays).
 *   - Return value: A3PO_OK or a negative a3po_error.  Argument errors are detected on the
 *     host before anything is launched; nothing is written in that case.
 *   - Conditions that only the device can see (a target index outside [0,V), a bounded wait
 *     that ran out) are OR-ed into the optional device word `status` (see A3PO_STATUS_*); the
 *     caller reads it after its own synchronisation.  An out-of-range target is clamped into
 *     range, never dereferenced.
 *   - N is the number of token rows.  Row-major layouts: hidden [N,H], W [V,H] (the LM head
 *     as stored by the model: one row per vocabulary entry), grad_hidden [N,H], grad_w [V,H].
 *   - `targets[t]` is the token whose probability is wanted at row t (the caller has already
 *     applied the next-token shift).
 *   - N = 0 is valid everywhere and is a no-op that still defines scalar outputs (loss = 0).
 */
#ifndef A3PO_H_
#define A3PO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  A3PO_OK = 0,
  A3PO_ERR_INVALID_ARG = -1,  /* NULL where a pointer is required, negative size, eps < 0 ...   */
  A3PO_ERR_UNSUPPORTED = -2,  /* dtype/shape/alignment the kernels do not handle                */
  A3PO_ERR_WORKSPACE = -3,    /* ws is NULL, misaligned or smaller than the minimum             */
  A3PO_ERR_CUDA = -4,         /* a CUDA runtime/driver call or a kernel launch failed           */
  A3PO_ERR_NO_DEVICE = -5,    /* no usable sm_100 device is current                             */
  A3PO_ERR_TOO_LARGE = -6     /* N exceeds the fixed scratch of a3po_loss_fwd_static            */
} a3po_error;

/* Storage type of hidden, W and grad_hidden.  Accumulation is always fp32. */
typedef enum { A3PO_F32 = 0, A3PO_BF16 = 1 } a3po_dtype;

/* Bits of the optional device status word. */
#define A3PO_STATUS_TARGET_OUT_OF_RANGE 1u /* some targets[t] was outside [0,V) and was clamped */
#define A3PO_STATUS_WAIT_TIMEOUT 2u        /* a bounded pipeline wait expired; results invalid  */
#define A3PO_STATUS_KEPT_RANGE 4u          /* keep-path only: some row's target probability is below
                                              about 1e-37, beyond what the kept ratios can express;
                                              that row's gradient contribution was dropped          */

/* Side outputs of the loss forward: the paper's per-step stability diagnostics
 * (importance-weight max/min, Fig. 5; number of clipped tokens, Fig. 6). */
typedef struct {
  int64_t n_valid;   /* M = number of tokens with mask != 0                                     */
  int64_t n_clipped; /* valid tokens whose clipped term is the strict minimum (zero gradient)   */
  float iw_max;      /* max over valid tokens of pi_prox/pi_behav (0 if M == 0)                 */
  float iw_min;      /* min over valid tokens of pi_prox/pi_behav (0 if M == 0)                 */
} a3po_stats;

const char* a3po_status_string(int code);

/* Library/ABI version: major*1000 + minor. */
int a3po_version(void);

/* --------------------------------------------------------------------------------------------
 * Policy forward, last stage (Sec. 2.2 "forward pass through the model"; Sec. 3: the engines
 * exchange token log-probabilities; Sec. 4.1: sampling temperature 1.0 => inv_temperature 1).
 *
 *   z[t,v]  = inv_temperature * sum_k hidden[t,k] * W[v,k]
 *   lse[t]  = log sum_v exp(z[t,v])
 *   logp[t] = z[t, targets[t]] - lse[t]
 *
 * The [N,V] logits are never written to memory: the contraction is fused with an online,
 * vocabulary-chunked log-sum-exp and the target gather.
 *
 * hidden [N,H], w [V,H]: dtype `dt`, 16-byte aligned, H % 8 == 0 for A3PO_BF16.
 * targets int32 [N].  row_mask uint8 [N] or NULL: rows with 0 report logp = lse = 0.
 * logp, lse: fp32 [N] outputs (lse is needed by the backward).
 * entropy: fp32 [N] or NULL; when given, receives the policy entropy -sum_v p_v log p_v of
 *          each row (the diagnostic of Fig. 4), computed in the same vocabulary sweep.
 * ws/ws_bytes: at least a3po_token_logprobs_min_workspace_bytes(N,H,V,dt,0).  With the larger
 * a3po_token_logprobs_workspace_bytes(N,H,V,dt,0) (bf16 inputs, row_mask given) the rows with
 * row_mask != 0 are gathered first and only they are multiplied; with less than that every row is
 * computed and the masked ones are discarded afterwards (same results, more work).
 * ------------------------------------------------------------------------------------------ */
size_t a3po_token_logprobs_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt, int is_bwd);

int a3po_token_logprobs_fwd(const void* hidden, const void* w, const int32_t* targets,
                            const uint8_t* row_mask, int64_t N, int H, int V, a3po_dtype dt,
                            float inv_temperature, float* logp, float* lse, float* entropy,
                            void* ws, size_t ws_bytes, uint32_t* status, void* stream);

/* --------------------------------------------------------------------------------------------
 * Backward of the above (the derivative of log-softmax + gather; no counterpart formula in the
 * paper, which leaves the backward to autograd):
 *
 *   dz[t,v]          = grad_logp[t] * (1[v == targets[t]] - exp(z[t,v] - lse[t])) * inv_temperature
 *   grad_hidden[t,:] = sum_v dz[t,v] * W[v,:]                      (dtype dt, [N,H], overwritten)
 *   grad_w[v,:]      = sum_t dz[t,v] * hidden[t,:]                 (fp32 [V,H])
 *
 * lse: the forward's output.  grad_logp fp32 [N]: rows with 0 contribute nothing.
 * accumulate_grad_w != 0 adds into grad_w (gradient accumulation over the mini-batches of a
 * training step, Sec. 4.1); 0 overwrites it.
 * dz is materialised only for a chunk of rows at a time inside `ws` (bf16 for A3PO_BF16);
 * the chunk length adapts to ws_bytes.  a3po_token_logprobs_workspace_bytes(...,1) returns
 * the size that lets the library use its preferred chunk AND gather the rows with a non-zero
 * grad_logp first (bf16 inputs), so that padding and clipped tokens cost nothing; with less
 * than that they are multiplied as zero rows (same results, more work).  The call fails with
 * A3PO_ERR_WORKSPACE below a3po_token_logprobs_min_workspace_bytes(...).
 * ------------------------------------------------------------------------------------------ */
size_t a3po_token_logprobs_min_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt, int is_bwd);

int a3po_token_logprobs_bwd(const void* hidden, const void* w, const int32_t* targets,
                            const float* lse, const float* grad_logp, int64_t N, int H, int V,
                            a3po_dtype dt, float inv_temperature, void* grad_hidden,
                            float* grad_w, int accumulate_grad_w, void* ws, size_t ws_bytes,
                            uint32_t* status, void* stream);

/* --------------------------------------------------------------------------------------------
 * Forward / backward pair that shares the softmax instead of recomputing the logits (bf16 inputs
 * only; no counterpart in the paper).  For callers whose forward and backward are separate calls,
 * as under an autograd engine:
 *
 *   a3po_token_logprobs_fwd_keep  = a3po_token_logprobs_fwd (same logp, lse, entropy; rows with
 *       row_mask 0 are skipped) that also fills `kept`.  For each row that took part it keeps the
 *       probability ratios q[t,v] = exp(z[t,v] - z[t,y_t]) = p[t,v] / p[t,y_t] in bf16 (a float
 *       ratio keeps bf16's relative precision whether the row is flat or peaked) and their sum
 *       s[t] over v != y_t, from which lse = z_y + log1p(s), logp = -log1p(s) and
 *       1 - p_y = s / (1 + s) follow without cancellation.
 *   a3po_token_logprobs_bwd_kept  = a3po_token_logprobs_bwd (same grad_hidden, grad_w within the
 *       gradient tolerance) that runs only the two gradient contractions, directly on q:
 *       dz[t,v] = a_t q'[t,v] with a_t = -grad_logp[t] inv_T / (1 + s[t]) and q'[t,y_t] = -s[t], so
 *       grad_hidden = diag(a) (q' W) and grad_w = q'^T (diag(a) hidden): 4 N V H flops instead of
 *       6 N V H for the backward, and no pass over an [N,V] matrix besides the contractions.
 *
 * `kept`: device buffer of a3po_kept_bytes(N, V) bytes (about 2 N V), 256-byte aligned, written by
 * the forward, read by the backward, which also writes the target entries q'[t,y_t] into it (the
 * same values on every call, so the backward may be repeated).  hidden, w, targets must be the
 * forward's; `lse` is accepted for symmetry with a3po_token_logprobs_bwd and not read.  Rows the
 * forward skipped get a zero gradient whatever their grad_logp.  A row whose target probability
 * is below about 1e-37 cannot be kept (A3PO_STATUS_KEPT_RANGE is raised, its contribution is
 * dropped).  Both calls return A3PO_ERR_UNSUPPORTED for shapes the tensor-core path does not take
 * (H % 8 != 0): use the plain pair then.  ws: at least the matching *_workspace_bytes.
 * ------------------------------------------------------------------------------------------ */
size_t a3po_kept_bytes(int64_t N, int V);
size_t a3po_token_logprobs_fwd_keep_workspace_bytes(int64_t N, int H, int V);
size_t a3po_token_logprobs_bwd_kept_workspace_bytes(int64_t N, int H, int V);

int a3po_token_logprobs_fwd_keep(const void* hidden, const void* w, const int32_t* targets,
                                 const uint8_t* row_mask, int64_t N, int H, int V,
                                 float inv_temperature, float* logp, float* lse, float* entropy,
                                 void* kept, size_t kept_bytes, void* ws, size_t ws_bytes,
                                 uint32_t* status, void* stream);

int a3po_token_logprobs_bwd_kept(const void* hidden, const void* w, const int32_t* targets,
                                 const float* lse, const float* grad_logp, void* kept,
                                 size_t kept_bytes, int64_t N, int H, int V, float inv_temperature,
                                 void* grad_hidden, float* grad_w, int accumulate_grad_w, void* ws,
                                 size_t ws_bytes, uint32_t* status, void* stream);

/* --------------------------------------------------------------------------------------------
 * A-3PO loss (Eq. 2 with the proximal policy of Eq. 3 and the coefficient of Eq. 4; argument
 * names follow Listing 1: behav_logp = old_logp, logp = logprobs, versions, current_version).
 *
 *   d_t     = current_version - versions[t]            (integer staleness)
 *   alpha_t = 1/d_t if d_t >= 1 else 1                 (d <= 0 gives 1, as the listing's where)
 *   lprox_t = alpha_t * behav_logp[t] + (1 - alpha_t) * logp[t]
 *   iw_t    = exp(lprox_t - behav_logp[t])             importance weight  pi_prox / pi_behav
 *   r_t     = exp(logp[t] - lprox_t)                   trust-region ratio pi_theta / pi_prox
 *   obj_t   = iw_t * min(r_t * adv[t], clip(r_t, 1-eps, 1+eps) * adv[t])
 *   loss    = - sum_t mask[t] * obj_t / max(M, 1),  M = sum_t mask[t]    (masked token mean)
 *
 * The kernels evaluate iw and r through the theorem's closed form r = w^alpha
 * (w = pi_theta/pi_behav), which is the same function with better fp32 conditioning.
 *
 * logp, behav_logp, adv: fp32 [N].  mask: uint8 [N] (0 = ignore; ignored tokens may hold any
 * bit pattern, NaN included: they are selected out, not multiplied).
 * versions: int32 [N] (one per token) when versions_per_seq == 0; int32 [B] (one per sequence)
 *   when versions_per_seq != 0, in which case cu_seqlens int32 [B+1] gives each sequence's row
 *   range [cu_seqlens[b], cu_seqlens[b+1]) with cu_seqlens[0] = 0 and cu_seqlens[B] = N.
 * clip_eps >= 0.
 * loss: fp32 device scalar.  stats: device struct or NULL.
 * The reduction is a fixed two-stage tree: results are bit-identical from run to run.  Where the
 * device supports cooperative launches the whole call is one kernel launch.
 * ws/ws_bytes: at least a3po_loss_workspace_bytes(N).
 * ------------------------------------------------------------------------------------------ */
size_t a3po_loss_workspace_bytes(int64_t N);

int a3po_loss_fwd(const float* logp, const float* behav_logp, const int32_t* versions,
                  int versions_per_seq, const int32_t* cu_seqlens, int B, int32_t current_version,
                  const float* adv, const uint8_t* mask, int64_t N, float clip_eps, float* loss,
                  a3po_stats* stats, void* ws, size_t ws_bytes, void* stream);

/* --------------------------------------------------------------------------------------------
 * dL/dlogp of the loss above.
 *
 *   act_t = 1 if r_t*adv_t <= clip(r_t)*adv_t (the unclipped term is the minimum) else 0
 *   detach_prox != 0 (default reading: the anchor is a constant, like the recomputed anchor of
 *   Sec. 2.2 which is "frozen"):      grad_logp[t] = -(gl * mask_t / M) * iw_t * adv_t * r_t * act_t
 *   detach_prox == 0 (differentiate through Eq. 3 too):
 *       grad_logp[t] = -(gl * mask_t / M) * ((1 - alpha_t) * obj_t + alpha_t * iw_t * adv_t * r_t * act_t)
 *
 * grad_loss: fp32 device scalar gl, or NULL for 1.
 * fwd_stats: the a3po_stats the forward wrote for the same inputs (supplies M), or NULL, in
 *   which case the mask is counted first (one extra byte per token of traffic).
 * grad_logp: fp32 [N] output; masked tokens get exactly 0.
 * ------------------------------------------------------------------------------------------ */
int a3po_loss_bwd(const float* logp, const float* behav_logp, const int32_t* versions,
                  int versions_per_seq, const int32_t* cu_seqlens, int B, int32_t current_version,
                  const float* adv, const uint8_t* mask, int64_t N, float clip_eps,
                  int detach_prox, const float* grad_loss, const a3po_stats* fwd_stats,
                  float* grad_logp, void* ws, size_t ws_bytes, void* stream);

/* Forward and backward in one pass over the inputs (mask counted first, then one stream that
 * reads 17 B/token and writes 4 B/token).  Outputs as in the two calls above; grad_loss = 1. */
int a3po_loss_fwd_bwd(const float* logp, const float* behav_logp, const int32_t* versions,
                      int versions_per_seq, const int32_t* cu_seqlens, int B,
                      int32_t current_version, const float* adv, const uint8_t* mask, int64_t N,
                      float clip_eps, int detach_prox, float* loss, a3po_stats* stats,
                      float* grad_logp, void* ws, size_t ws_bytes, void* stream);

/* --------------------------------------------------------------------------------------------
 * The decoupled clipped loss of Eq. 2 with an EXPLICIT proximal policy: the baseline the paper
 * calls "recompute" (Sec. 2.2: log pi_prox comes from an extra forward pass and is frozen), and,
 * with prox_logp = behav_logp, the coupled PPO-clip loss of Eq. 1 ("sync").  Same streaming
 * kernel as a3po_loss_fwd_bwd with the interpolation replaced by a load:
 *
 *   iw_t  = exp(prox_logp[t] - behav_logp[t]),   r_t = exp(logp[t] - prox_logp[t])
 *   obj_t = iw_t * min(r_t * adv[t], clip(r_t, 1-eps, 1+eps) * adv[t])
 *   loss  = - sum_t mask[t] * obj_t / max(M, 1)
 *   grad_logp[t] = -(mask_t / M) * iw_t * adv_t * r_t * act_t        (the anchor is a constant)
 *
 * prox_logp: fp32 [N].  grad_logp may be NULL (forward only).  Other arguments, outputs,
 * workspace and error codes as a3po_loss_fwd_bwd.
 * ------------------------------------------------------------------------------------------ */
int a3po_decoupled_loss_fwd_bwd(const float* logp, const float* behav_logp, const float* prox_logp,
                                const float* adv, const uint8_t* mask, int64_t N, float clip_eps,
                                float* loss, a3po_stats* stats, float* grad_logp, void* ws,
                                size_t ws_bytes, void* stream);

/* --------------------------------------------------------------------------------------------
 * Helpers for data-parallel training over sequences (no counterpart in the paper, which states E_t
 * of Eq. 2 for one batch).  The path is per token except the masked mean, so a job that shards its
 * sequences over ranks gets the whole-job loss and gradients from per-rank calls as
 *     L = sum_r (M_r / M) L_r,     grad = sum_r (M_r / M) grad_r,      M = sum_r M_r,
 * where L_r, grad_r are what rank r computes with its local mean.  a3po_mask_count gives M_r before
 * the step (the mask is an input), the caller all-reduces it, a3po_dp_loss_scale turns the two
 * counts into the weight M_r / M, and a3po_train_step takes that weight as `loss_scale`, so its
 * gradients come out already weighted and one sum all-reduce of grad_w (and of the weighted loss)
 * finishes the job; grad_hidden and grad_logp stay local.
 *
 * a3po_mask_count: *count (int64, device) = number of non-zero mask bytes; ws of
 *   a3po_mask_count_workspace_bytes() bytes.
 * a3po_dp_loss_scale: *scale = M_local / M_global (0 if M_global == 0), all device scalars; when
 *   loss_local is given, *weighted_loss = *scale * *loss_local as well.
 * ------------------------------------------------------------------------------------------ */
size_t a3po_mask_count_workspace_bytes(void);
int a3po_mask_count(const uint8_t* mask, int64_t N, int64_t* count, void* ws, size_t ws_bytes, void* stream);
int a3po_dp_loss_scale(const int64_t* m_local, const int64_t* m_global, const float* loss_local,
                       float* scale, float* weighted_loss, void* stream);

/* --------------------------------------------------------------------------------------------
 * GRPO advantages (Sec. 4.1: "estimate advantages using group reward normalization"; the paper
 * gives no formula, the customary one is used).  Sequences come in consecutive groups of
 * `group_size` responses to the same prompt:
 *
 *   A_i = (R_i - mean_group) / (std_group + norm_eps)        population standard deviation
 *   adv[t] = A_i for every row t of sequence i, i.e. cu_seqlens[i] <= t < cu_seqlens[i+1]
 *
 * rewards fp32 [B], cu_seqlens int32 [B+1] (cu_seqlens[0] = 0, cu_seqlens[B] = N), B a multiple
 * of group_size, adv fp32 [N] output.  ws: at least a3po_grpo_workspace_bytes(B).
 * ------------------------------------------------------------------------------------------ */
size_t a3po_grpo_workspace_bytes(int B);

int a3po_grpo_advantages(const float* rewards, int B, int group_size, const int32_t* cu_seqlens,
                         int64_t N, float norm_eps, float* adv, void* ws, size_t ws_bytes,
                         void* stream);

/* --------------------------------------------------------------------------------------------
 * Self-test of the bounded waits the pipelined kernels rely on (no counterpart in the paper).
 * Launches a one-warp kernel that waits on a barrier nothing ever signals; after timeout_ms
 * (1..2000) the wait gives up and ORs A3PO_STATUS_WAIT_TIMEOUT into *status (device word),
 * which is what a stuck pipeline stage does instead of hanging the GPU.
 * ------------------------------------------------------------------------------------------ */
int a3po_selftest_wait_timeout(uint32_t* status, unsigned timeout_ms, void* stream);

/* --------------------------------------------------------------------------------------------
 * a3po_loss_fwd for callers that have no way to hand over a workspace (the paper has no
 * counterpart: this is a packaging variant, the arithmetic is a3po_loss_fwd's).
 *
 * Who needs it: code that runs where device memory cannot be obtained at call time — a hook
 * inside a host framework whose memory pool is the only permitted allocator and is not exposed
 * to the hook, a latency-critical loop in which an allocation (an implicit device-wide
 * synchronisation) is forbidden, or a process whose device memory has been carved up in advance
 * and where cudaMalloc simply fails.  Such a caller still owns its inputs and outputs; what it
 * lacks is the few megabytes of scratch the loss kernels reduce through.
 *
 * Here that scratch is a fixed array inside the library's device image (about 4.2 MiB, sized
 * for A3PO_LOSS_FWD_STATIC_MAX_TOKENS tokens).  Every GPU on which the library is loaded holds
 * it from load until the process exits, whether or not this function is ever called.  The
 * function calls no cudaMalloc / cudaFree and no allocating library routine (with the optional
 * per-kernel profile left off, which is the default, it creates no CUDA objects at all).
 *
 * Arguments, outputs and error codes are those of a3po_loss_fwd without ws / ws_bytes, plus:
 *   - N > A3PO_LOSS_FWD_STATIC_MAX_TOKENS returns A3PO_ERR_TOO_LARGE before anything is
 *     launched or written; use a3po_loss_fwd with a caller workspace for larger batches.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  That first call should be made before any stream capture begins.
 *   - All calls on one device share the one array.  Nothing in it has to be zero on entry: a call
 *     reads only words it has written itself, so the previous call's leftovers are harmless.
 *     But two calls whose kernels overlap on the GPU (different streams, or different host
 *     threads without ordering) race on it and corrupt each other's result: serialise them.
 * ------------------------------------------------------------------------------------------ */
#define A3PO_LOSS_FWD_STATIC_MAX_TOKENS (1 << 20)

int a3po_loss_fwd_static(const float* logp, const float* behav_logp, const int32_t* versions,
                         int versions_per_seq, const int32_t* cu_seqlens, int B,
                         int32_t current_version, const float* adv, const uint8_t* mask, int64_t N,
                         float clip_eps, float* loss, a3po_stats* stats, void* stream);

/* --------------------------------------------------------------------------------------------
 * One whole training-step pass with every buffer on the device (no counterpart in the paper):
 *   logp, lse [, entropy]  = token_logprobs_fwd(hidden, w, targets, row_mask = mask)
 *   loss, stats, grad_logp = loss_fwd_bwd(logp, behav_logp, versions (per token), ...)   detach_prox = 1
 *   grad_hidden, grad_w    = token_logprobs_bwd(..., lse, grad_logp)
 * with the same results as the three calls.  For bf16 inputs and a workspace of at least
 * a3po_train_step_workspace_bytes(...) the step does not recompute the LM head in the backward
 * (6 N V H flops instead of 8 N V H): the rows with mask != 0 are gathered once (their number M
 * is then known on the device), and per chunk of those rows the forward keeps the softmax as
 * bf16 probability ratios (see a3po_token_logprobs_fwd_keep), the loss forward + backward runs
 * on the chunk's log-probs, and the two gradient contractions run on the kept ratios.  The
 * workspace holds one chunk of ratios at a time (chunk x V x 2 bytes; the recommended size is
 * for chunks of 65,536 rows, about 20 GB at V = 151,936, and a larger workspace gives larger
 * chunks) plus a gathered copy of hidden.  With a smaller workspace (at least
 * a3po_train_step_min_workspace_bytes) or fp32 inputs the three calls are made as they are.
 * logp, lse, grad_logp: fp32 [N] outputs.  entropy: fp32 [N] or NULL (policy entropy per row,
 * Fig. 4).  loss_scale: fp32 device scalar or NULL (= 1): every gradient (grad_logp, grad_hidden,
 * grad_w) is multiplied by it, the reported loss is not; data-parallel callers pass M_local /
 * M_global (see a3po_dp_loss_scale).  Other arguments as in the individual calls.
 * ------------------------------------------------------------------------------------------ */
size_t a3po_train_step_min_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt);
size_t a3po_train_step_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt);

int a3po_train_step(const void* hidden, const int32_t* targets, const float* behav_logp,
                    const int32_t* versions, const float* adv, const uint8_t* mask, int64_t N, int H,
                    int V, a3po_dtype dt, int32_t current_version, float clip_eps,
                    float inv_temperature, const void* w, float* grad_w, int accumulate_grad_w,
                    void* grad_hidden, float* logp, float* lse, float* entropy, float* grad_logp,
                    float* loss, a3po_stats* stats, const float* loss_scale, void* ws, size_t ws_bytes,
                    uint32_t* status, void* stream);

/* --------------------------------------------------------------------------------------------
 * The same pass with per-step inputs in HOST memory (no counterpart in the paper; this is the
 * end-to-end form of the call above):
 *   copies hidden, targets, behav_logp, versions, adv, mask host->device, runs a3po_train_step,
 *   copies loss + stats back.
 * Of `hidden`, only the runs of rows with mask != 0 are copied when the step keeps its softmax
 * (it reads no other row; the rest of the staged copy is then undefined); every row is copied
 * when the workspace or the shape sends the step down the recomputing calls.
 * h_* are host pointers (pinned memory recommended; pageable works but serialises); h_mask is
 * read by the host during the call.
 * d_w, d_grad_w (accumulated into when accumulate_grad_w != 0), d_grad_hidden ([N,H] dt) and
 * d_stage/d_ws are device buffers.  d_stage needs a3po_train_step_stage_bytes(N,H,dt) bytes and
 * d_ws a3po_train_step_workspace_bytes(N,H,V,dt).  h_loss (float) and h_stats are host outputs,
 * valid after the caller synchronises `stream`.
 * ------------------------------------------------------------------------------------------ */
size_t a3po_train_step_stage_bytes(int64_t N, int H, a3po_dtype dt);

int a3po_train_step_host(const void* h_hidden, const int32_t* h_targets, const float* h_behav_logp,
                         const int32_t* h_versions, const float* h_adv, const uint8_t* h_mask,
                         int64_t N, int H, int V, a3po_dtype dt, int32_t current_version,
                         float clip_eps, float inv_temperature, const void* d_w, float* d_grad_w,
                         int accumulate_grad_w, void* d_grad_hidden, void* d_stage,
                         size_t stage_bytes, void* d_ws, size_t ws_bytes, float* h_loss,
                         a3po_stats* h_stats, uint32_t* d_status, void* stream);

/* Bytes the host entries of this library have copied host->device in the calling process since
 * load (monotonic; for transfer accounting in benchmarks). */
int64_t a3po_host_to_device_bytes(void);

/* Number of kernels this library has launched in the calling process since load
 * (monotonic; for launch accounting in benchmarks). */
int64_t a3po_kernel_launch_count(void);

/* --------------------------------------------------------------------------------------------
 * Optional per-kernel timing (no counterpart in the paper).  While enabled, every kernel the
 * library launches is bracketed by a pair of CUDA events recorded on the launch stream.
 * a3po_profile_read waits for the recorded events, returns up to max_entries (kernel id,
 * milliseconds) pairs in launch order, and clears the record list; a3po_kernel_name maps an id
 * to a static string.  Host-side state is process-global and mutex-protected.  Leave it off
 * for production use: each launch costs two extra event records.
 * ------------------------------------------------------------------------------------------ */
int a3po_profile_enable(int on);
int a3po_profile_read(int max_entries, int* kernel_ids, float* milliseconds, int* count);
const char* a3po_kernel_name(int kernel_id);

#ifdef __cplusplus
}
#endif
#endif /* A3PO_H_ */
