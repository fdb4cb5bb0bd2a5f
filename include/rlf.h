/*
 * rlf.h -- C ABI of the B200 (sm_100a) GRPO policy-update loss path.
 *
 * The path, in call order for one training micro-batch of packed multi-turn
 * tool-use responses:
 *     rlf_build_loss_mask  ->  rlf_group_advantage  ->
 *     rlf_grpo_logp_loss_fwd_bwd   (logits materialised by the caller)   or
 *     rlf_fused_lmhead_grpo        (logits formed on the fly from hidden states)
 *
 * Conventions that hold for every entry point unless stated otherwise:
 *   - Every pointer is DEVICE memory owned by the caller and valid on the
 *     current device until the work queued on `stream` has finished.  The
 *     library allocates nothing and never synchronises: it validates
 *     arguments on the host, queues kernels (and small memsets) on `stream`,
 *     and returns.  The one exception is rlf_grpo_step_host, which takes HOST
 *     buffers and ends with a stream synchronisation.
 *   - State: a compute call leaves nothing behind that a later call depends
 *     on.  What the library does keep is (a) per-device caches of facts that
 *     never change while the process lives (the architecture check, kernel
 *     attributes and occupancy, the device address of the *_static entry
 *     point's built-in scratch), filled on first use under a lock, and (b) the
 *     PROCESS-WIDE tuning knobs set by the rlf_tune_* calls.  A knob changes
 *     every later compute call of every thread (rlf_tune_logits_kernel can
 *     make a later call return RLF_ERR_UNSUPPORTED for a shape that cannot
 *     hold a row); the knobs are plain atomics, so set them before compute
 *     calls start on other threads, not beside them.  Compute calls themselves
 *     are re-entrant.
 *   - `stream` is a CUDA stream handle (cudaStream_t); NULL is the default stream.
 *   - Host-detectable problems return a negative rlf_status before anything is
 *     queued.  Problems only visible on the device (a target id outside the
 *     vocabulary, a malformed cu_seqlens, a non-finite row) OR a bit into
 *     *dev_status (caller-owned int32 on the device, may be NULL; never
 *     cleared by the library) and neutralise the offending row: it gets loss
 *     weight 0 and an all-zero gradient.  Kernels never trap or assert.
 *   - Row r of logits / hidden predicts token ids[r]; the caller has already
 *     applied the next-token shift.  Rows [cu_seqlens[b], cu_seqlens[b+1]) belong to response b.
 *   - There is no CPU fallback: on a device that is not compute capability
 *     10.x every compute entry point returns RLF_ERR_ARCH.
 */
#ifndef RLF_H_
#define RLF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RLF_OK = 0,
    RLF_ERR_NULL = -1,      /* a required pointer is NULL */
    RLF_ERR_SHAPE = -2,     /* a size is negative / zero where it may not be / inconsistent */
    RLF_ERR_ALIGN = -3,     /* a pointer or stride violates the stated alignment */
    RLF_ERR_DTYPE = -4,     /* unknown rlf_dtype */
    RLF_ERR_WORKSPACE = -5, /* workspace NULL, misaligned or smaller than rlf_workspace_bytes() */
    RLF_ERR_ARCH = -6,      /* current device is not sm_100 */
    RLF_ERR_CUDA = -7,      /* a CUDA runtime call failed (launch, memset, copy) */
    RLF_ERR_UNSUPPORTED = -8, /* valid request outside what this library implements */
    RLF_ERR_TOO_LARGE = -9   /* more tokens than the built-in scratch of a *_static entry point holds */
} rlf_status;

typedef enum { RLF_BF16 = 0, RLF_F32 = 1 } rlf_dtype;

/* bits OR-ed into *dev_status by kernels */
#define RLF_DEV_BAD_TARGET 1   /* ids[r] outside [0, V) */
#define RLF_DEV_BAD_SEQ 2      /* cu_seqlens not monotone / outside [0, T], or seq_id outside [0, B) */
#define RLF_DEV_NONFINITE 4    /* a row's log-sum-exp or log-prob is not finite */
#define RLF_DEV_TIMEOUT 8      /* a bounded device-side wait gave up */

/* selectors for rlf_workspace_bytes */
#define RLF_FN_LOGP_LOSS 3
#define RLF_FN_FUSED_LMHEAD 4
#define RLF_FN_LOGP_ENTROPY 5
#define RLF_FN_FUSED_LOGP_ENTROPY 6

typedef struct CUstream_st *rlf_stream_t;

/*
 * Loss mask from observation markers.  (Paper Sec. 2.2: observation tokens are
 * tool output appended to the trajectory and take no part in the loss; Sec.
 * 2.3.2: a loss mask is set over tool results.)
 *
 * A span runs from a token equal to `open_id` to the next token equal to
 * `close_id` in the same response, both markers included; every token of a
 * span gets mask 0, every other token 1.  A close marker outside a span is an
 * ordinary token, an open marker inside a span changes nothing, a span that is
 * not closed runs to the end of its response, and the state resets at every
 * response start.  If `valid` is given the result is AND-ed with valid[t] != 0.
 *
 *   ids         [T] int32   target token ids (packed responses)
 *   cu_seqlens  [B+1] int32 response boundaries, cu_seqlens[0] = 0, cu_seqlens[B] = T
 *   valid       [T] uint8 or NULL
 *   mask_out    [T] uint8   written for every t (tokens outside every response get 0)
 *   seq_id_out  [T] int32 or NULL: response index of each token (-1 outside every response)
 *   n_out       [1] int64   number of tokens with mask 1 (overwritten)
 * T = 0 and B = 0 are valid.  A non-monotone or out-of-range cu_seqlens sets RLF_DEV_BAD_SEQ and
 * the affected response is clipped to [0, T).
 */
rlf_status rlf_build_loss_mask(const int32_t *ids, const int32_t *cu_seqlens, int32_t B, int64_t T,
                               int32_t open_id, int32_t close_id, const uint8_t *valid,
                               uint8_t *mask_out, int32_t *seq_id_out, int64_t *n_out,
                               int32_t *dev_status, rlf_stream_t stream);

/*
 * Number of responses that carry loss: those with at least one token of mask 1.  (Paper Sec. 2.3.2:
 * the loss is taken over the model's own tokens; a response that is all tool feedback, or cut to
 * nothing, carries none.)  It is the denominator of the sequence-mean aggregation of the *_obj entry
 * points (their `denom`), which a caller needs on its own when one batch is spread over several calls
 * or several GPUs: each part counts its responses and the counts are added.
 *   mask [T] uint8;  cu_seqlens [B+1] int32;  *count_out int64 on the device (overwritten)
 * A malformed cu_seqlens sets RLF_DEV_BAD_SEQ and the response is clipped to [0, T).  B = 0 is valid.
 */
rlf_status rlf_count_live_responses(const uint8_t *mask, const int32_t *cu_seqlens, int32_t B, int64_t T,
                                    int64_t *count_out, int32_t *dev_status, rlf_stream_t stream);

/*
 * Group-relative outcome advantage.  (Paper Sec. 2.3.2 / Fig. 4 name GRPO as
 * the algorithm; the formula is the standard group normalisation.)
 *     A_i = (r_i - mean_g) / (std_g + eps),  g = group of response i
 * std_g divides by n-1 if `unbiased_std` else by n; a group with one member or
 * zero spread gets A = 0.  Sums are accumulated in fp64 in index order.
 *
 *   rewards   [B] fp32
 *   group_id  [B] int32 in [0, g_or_num_groups), or NULL: response i is in group i / g_or_num_groups
 *   g_or_num_groups  number of groups if group_id is given, else the group size G
 *   adv_out   [B] fp32
 * A group_id outside its range sets RLF_DEV_BAD_SEQ and gives that response A = 0.
 */
rlf_status rlf_group_advantage(const float *rewards, const int32_t *group_id, int32_t B,
                               int32_t g_or_num_groups, float eps, int unbiased_std,
                               float *adv_out, int32_t *dev_status, rlf_stream_t stream);

/*
 * Rule reward.  (Paper Eq. 1: R_rule = sum_i w_i r_i over the n rule dimensions, e.g. call-format
 * validity, task completion, efficiency.)  The result feeds rlf_group_advantage as `rewards`.
 * Scores that a judge model (Eq. 2) or a verification tool (Eq. 3) produced elsewhere enter the same
 * way, as further columns with weights of their own.
 *   scores [B, n] fp32 row-major;  weights [n] fp32;  reward_out [B] fp32 (fp64 accumulation)
 */
rlf_status rlf_rule_reward(const float *scores, const float *weights, int32_t B, int32_t n,
                           float *reward_out, rlf_stream_t stream);

/*
 * KL penalty folded into the outcome reward instead of the loss (an objective variant of the GRPO /
 * PPO-style update that the paper names in Sec. 2.3.1 and Sec. 2.3.2; the paper prints no formula,
 * this is the usual form).  Call it between the reward and rlf_group_advantage, and run the loss with
 * beta_kl = 0:
 *     R'_b = R_b - beta * sum_{t in response b} mask[t] k(d_t),   d_t = old_logp[t] - ref_logp[t]
 *     kl_kind RLF_KL_K1: k = d;   RLF_KL_K2: k = d^2 / 2;   RLF_KL_K3: k = exp(-d) + d - 1
 * Sums are taken in fp64 in a fixed order (results are run-to-run identical).
 *
 *   rewards     [B] fp32;  old_logp, ref_logp [T] fp32;  mask [T] uint8
 *   cu_seqlens  [B+1] int32: response b owns tokens cu_seqlens[b] .. cu_seqlens[b+1]-1
 *   reward_out  [B] fp32 (may be the same buffer as rewards)
 *   kl_seq_out  [B] fp32 or NULL: the summed estimate of each response
 * A malformed cu_seqlens sets RLF_DEV_BAD_SEQ and the response is clipped to [0, T).  An unknown
 * kl_kind returns RLF_ERR_UNSUPPORTED.  B = 0 and T = 0 are valid.
 */
#define RLF_KL_K1 0
#define RLF_KL_K2 1
#define RLF_KL_K3 2
rlf_status rlf_kl_in_reward(const float *rewards, const float *old_logp, const float *ref_logp,
                            const uint8_t *mask, const int32_t *cu_seqlens, int32_t B, int64_t T,
                            float beta, int kl_kind, float *reward_out, float *kl_seq_out,
                            int32_t *dev_status, rlf_stream_t stream);

/*
 * Fused log-prob + clipped-ratio + k3-KL loss, forward and backward, over
 * materialised logits.  (Paper Sec. 2.2: the policy pi_theta(a | s_t); Sec.
 * 2.3.1: PPO-style update of the RL trainer; Sec. 2.3.2: GRPO with the loss
 * mask.  Formulas are the textbook ones.)  Per row t with y = ids[t]:
 *     lse = log sum_v exp z[t,v];   logp = z[t,y] - lse
 *     rho = exp(logp - old_logp[t]);  A = adv[seq_id[t]]
 *     pg  = -min(rho A, clip(rho, 1-eps_clip, 1+eps_clip) A)
 *     d   = ref_logp[t] - logp;  kl = exp(d) - d - 1
 *     N   = *denom if denom != NULL else sum_t mask[t];   Nd = max(N, 1)
 *     loss_out = { sum mask (pg + beta kl), sum mask pg, sum mask kl, sum mask clipped } / Nd
 *     grad_logits[t,v] = d loss_out[0] / d z[t,v] = c_t (softmax(z[t,:])[v] - 1[v = y]),
 *         c_t = -(mask[t]/Nd) (dpg/dlogp + beta (1 - exp d)),
 *         dpg/dlogp = 0 where the clipped branch is active (A>0, rho>1+eps or A<0, rho<1-eps), else -A rho.
 *     The target column is formed as -c_t S'/S, S' the row's exponential sum over the other columns,
 *     so it keeps its relative accuracy when softmax[y] rounds to one.
 * Each logits row is read from HBM once and grad written once; max / sum are
 * accumulated in fp32, the token-level loss terms are summed in fp64 in a fixed order
 * (results are run-to-run identical).
 *
 *   logits       [T, V] dt, row r starts at element r * row_stride (row_stride >= V)
 *   ids          [T] int32;  seq_id [T] int32 in [0, B);  adv [B] fp32
 *   old_logp, ref_logp [T] fp32;  mask [T] uint8
 *   denom        [1] int64 on the device, or NULL.  Pass the global token count when a batch is
 *                split over several calls so that the calls' losses and gradients add up.
 *   logp_out     [T] fp32, written for every row (masked or not)
 *   loss_out     [4] fp64
 *   grad_logits  [T, V] dt with the same row_stride, or NULL (forward only).  May be the same
 *                buffer as logits (in place).  Masked rows are written as zeros.
 *   workspace    rlf_workspace_bytes(RLF_FN_LOGP_LOSS, T, V, 0, dt) bytes, 256-byte aligned;
 *                contents need not be initialised and are overwritten.
 * Fast path: dt = RLF_BF16, V a multiple of 8, row_stride a multiple of 8, both bases 16-byte
 * aligned.  Anything else (fp32 logits, odd V, unaligned rows) takes a slower general kernel.
 * T = 0 is valid (loss_out = 0).
 */
rlf_status rlf_grpo_logp_loss_fwd_bwd(const void *logits, rlf_dtype dt, int64_t T, int32_t V,
                                      int64_t row_stride, const int32_t *ids,
                                      const int32_t *seq_id, const float *adv, int32_t B,
                                      const float *old_logp, const float *ref_logp,
                                      const uint8_t *mask, float eps_clip, float beta_kl,
                                      const int64_t *denom, float *logp_out, double *loss_out,
                                      void *grad_logits, void *workspace, size_t workspace_bytes,
                                      int32_t *dev_status, rlf_stream_t stream);

/*
 * rlf_grpo_logp_loss_fwd_bwd with the objective's common variants.  (The paper names GRPO and a
 * PPO-style update, Sec. 2.3, without printing the objective; these are the usual alternatives.)
 *   clip range     clip(rho, 1 - eps_clip_low, 1 + eps_clip_high)
 *   aggregation 0  masked token mean over the call (N = *denom or the sum of mask), as above
 *   aggregation 1  mean over responses of each response's masked token mean: token t of response b
 *                  has weight mask[t] / (n_b S), n_b = live tokens of b, S = *denom if denom != NULL
 *                  (number of responses of the whole batch when it is split over calls), else the
 *                  number of responses with n_b > 0 in this call.  Needs B <= T + 1.
 * loss_out[k] = sum of weight x {pg + beta kl, pg, kl, clipped}; grad_logits scales accordingly.
 * All other arguments, the workspace size and the error behaviour are those of
 * rlf_grpo_logp_loss_fwd_bwd, which equals this call with eps_clip_low = eps_clip_high, aggregation 0.
 */
rlf_status rlf_grpo_logp_loss_fwd_bwd_obj(const void *logits, rlf_dtype dt, int64_t T, int32_t V,
                                          int64_t row_stride, const int32_t *ids, const int32_t *seq_id,
                                          const float *adv, int32_t B, const float *old_logp,
                                          const float *ref_logp, const uint8_t *mask,
                                          float eps_clip_low, float eps_clip_high, float beta_kl,
                                          int aggregation, const int64_t *denom, float *logp_out,
                                          double *loss_out, void *grad_logits, void *workspace,
                                          size_t workspace_bytes, int32_t *dev_status,
                                          rlf_stream_t stream);

/*
 * rlf_grpo_logp_loss_fwd_bwd that neither reads nor computes rows without loss weight.  (Paper
 * Sec. 2.2 / Sec. 2.3.2: observation tokens take no part in the loss; in multi-turn tool-use batches
 * they are a large share of all tokens, so their logits rows need not be touched at all.)
 * Rows with mask 0 (and rows neutralised for a bad target / sequence id) are skipped:
 *   - logp_out[t] of a skipped row is NaN;
 *   - its grad_logits row is written as zeros if zero_masked_grad != 0, and left untouched
 *     otherwise (for callers that zero the buffer themselves or never read those rows);
 *   - loss_out and the live rows' logp / grad are exactly those of rlf_grpo_logp_loss_fwd_bwd.
 * Arguments otherwise as for rlf_grpo_logp_loss_fwd_bwd; same workspace size.  HBM traffic is
 * 4 V bytes per live token plus 2 V per skipped token that is zero-filled.  Logits that do not
 * qualify for the fast path are processed in full by the general kernel (same results).
 */
rlf_status rlf_grpo_logp_loss_fwd_bwd_skip_masked(const void *logits, rlf_dtype dt, int64_t T, int32_t V,
                                                  int64_t row_stride, const int32_t *ids,
                                                  const int32_t *seq_id, const float *adv, int32_t B,
                                                  const float *old_logp, const float *ref_logp,
                                                  const uint8_t *mask, float eps_clip, float beta_kl,
                                                  const int64_t *denom, float *logp_out,
                                                  double *loss_out, void *grad_logits,
                                                  int zero_masked_grad, void *workspace,
                                                  size_t workspace_bytes, int32_t *dev_status,
                                                  rlf_stream_t stream);

/*
 * Forward-only log-prob of given target tokens, and the entropy of each row's distribution: the pass
 * that produces old_logp / ref_logp for the update above (the behaviour and reference policies of
 * the PPO-style update, paper Sec. 2.3.1; the policy pi_theta(a | s_t) of Sec. 2.2).  Per row t:
 *     logp[t]    = z[t, ids[t]] - log sum_v exp z[t, v]
 *     entropy[t] = - sum_v p_v log p_v,  p = softmax(z[t, :])      (terms with p_v = 0 contribute 0)
 * Each logits row is read from HBM once (2 V bytes per token at bf16); nothing else of size T x V
 * is touched.  Same fast-path conditions, general fallback and device status bits as
 * rlf_grpo_logp_loss_fwd_bwd; a row with a target outside [0, V) or a non-finite log-sum-exp gets
 * NaN.  workspace: rlf_workspace_bytes(RLF_FN_LOGP_ENTROPY, T, V, 0, dt) bytes select the streaming
 * form (rows cut into chunks whose partial statistics a second kernel merges); with only
 * rlf_workspace_bytes(RLF_FN_LOGP_LOSS, ...) bytes the row-per-cluster form runs instead.
 *   logits [T, V] dt with row_stride;  ids [T] int32;  logp_out [T] fp32;  entropy_out [T] fp32 or NULL
 */
rlf_status rlf_logp_entropy_fwd(const void *logits, rlf_dtype dt, int64_t T, int32_t V, int64_t row_stride,
                                const int32_t *ids, float *logp_out, float *entropy_out, void *workspace,
                                size_t workspace_bytes, int32_t *dev_status, rlf_stream_t stream);

/*
 * rlf_grpo_logp_loss_fwd_bwd without a workspace argument, for callers that cannot allocate.
 * (The paper has no counterpart: this is a packaging variant of the entry point above.)
 *
 * Who needs it: code that sits where device allocation is not an option -- a training-loop thread
 * that must not trigger the device-wide synchronisation cudaMalloc / cudaFree imply, a process
 * whose framework has already claimed all device memory for its own pool, or a plug-in that has
 * no handle on the host framework's allocator.  Such a caller still owns every input and output
 * buffer; only the kernels' scratch (token records and partial sums) moves into the library.
 *
 * The scratch is a fixed array in the library's device image, RLF_STATIC_MAX_TOKENS tokens large
 * (about 2.9 MB, the workspace of a batch of that size; every GPU that loads the library holds it
 * until the process exits).  This call
 * allocates nothing, on the device or through any library: T > RLF_STATIC_MAX_TOKENS returns
 * RLF_ERR_TOO_LARGE before anything is queued.  All other arguments, results and errors are
 * those of rlf_grpo_logp_loss_fwd_bwd, and the same kernels run.
 *
 * The first call on each device looks the array's device address up (one runtime query, made with
 * that device current, its result checked and remembered); make that first call outside any stream
 * capture.  Every call on a device uses the same array: it keeps the previous call's contents,
 * which is harmless (each call rewrites what it reads and zeroes its token counter itself), but
 * two calls whose kernels overlap on the GPU -- different streams without an ordering between
 * them -- race on it.  Serialise such calls or give the second one its own workspace through
 * rlf_grpo_logp_loss_fwd_bwd.
 */
#define RLF_STATIC_MAX_TOKENS 65536
rlf_status rlf_grpo_logp_loss_fwd_bwd_static(const void *logits, rlf_dtype dt, int64_t T, int32_t V,
                                             int64_t row_stride, const int32_t *ids,
                                             const int32_t *seq_id, const float *adv, int32_t B,
                                             const float *old_logp, const float *ref_logp,
                                             const uint8_t *mask, float eps_clip, float beta_kl,
                                             const int64_t *denom, float *logp_out,
                                             double *loss_out, void *grad_logits,
                                             int32_t *dev_status, rlf_stream_t stream);

/*
 * Same loss with the logits formed on the fly, z = hidden W^T, so that they
 * never reach HBM.  (Paper Sec. 2.2: pi_theta is the language model's output
 * head; the fusion itself is this library's design.)  The backward runs over the
 * unmasked rows only (the others have zero gradient) and returns
 *     grad_hidden[t,:] = sum_v grad_z[t,v] W[v,:]       (bf16)
 *     grad_W[v,:]      = sum_t grad_z[t,v] hidden[t,:]  (fp32; added to the buffer if accumulate_grad_W)
 *
 *   hidden [T, D] bf16 row-major;  W [V, D] bf16 row-major; both 16-byte aligned, D a multiple of
 *               64 and V a multiple of 8 (else RLF_ERR_SHAPE)
 *   per-token arguments, denom, logp_out, loss_out: as for rlf_grpo_logp_loss_fwd_bwd
 *   grad_hidden [T, D] bf16 or NULL;  grad_W [V, D] fp32 or NULL (both NULL: forward only)
 *   workspace   rlf_workspace_bytes(RLF_FN_FUSED_LMHEAD, T, V, D, RLF_BF16) bytes, 256-byte aligned.
 *               It holds per-token records and partial sums and, for the backward, a copy of hidden
 *               with the unmasked rows gathered first, one chunk of those rows times their row
 *               factors, and one chunk of min(T, 18944) rows by V (rounded up to whole 256-column
 *               tiles) of bf16, stored in blocks of 128 rows x 64 columns (5.8 GB at V = 151936,
 *               T >= 18944): the forward sweep of a chunk of unmasked rows leaves exp(z - rho_t)
 *               there, rho_t a per-row reference fixed before the sweep (the row's fp32 target logit
 *               plus 32: bf16 has fp32's exponent range, so the entries that matter stay normal
 *               numbers), and the two gradient contractions consume it with the per-row factor
 *               c_t exp(rho_t - lse_t) applied in fp32 (grad_hidden) or to the hidden rows (grad_W).
 *               A chunk with a row whose reference proves unusable (target log-prob below about -78)
 *               is redone on the device with exponentials against per-tile maxima and one rescaling
 *               pass over the scratch.  The logits themselves are never stored.
 * Tensor-core contractions are bf16 x bf16 with fp32 accumulation in tensor memory; the stored
 * exponentials are rounded to bf16 once, the scaled hidden rows of grad_W once more.  The contraction
 * launches are persistent kernels of one CTA per SM whose workers meet on a counter in the workspace
 * (see rlf_tune_lmhead_pacing); they are fastest with the GPU to themselves.  Waits inside the kernels
 * are bounded: if one of the data waits runs out, RLF_DEV_TIMEOUT is set in *dev_status and the
 * outputs are not valid.
 */
rlf_status rlf_fused_lmhead_grpo(const void *hidden, const void *W, int64_t T, int32_t D, int32_t V,
                                 const int32_t *ids, const int32_t *seq_id, const float *adv,
                                 int32_t B, const float *old_logp, const float *ref_logp,
                                 const uint8_t *mask, float eps_clip, float beta_kl,
                                 const int64_t *denom, float *logp_out, double *loss_out,
                                 void *grad_hidden, float *grad_W, int accumulate_grad_W,
                                 void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                 rlf_stream_t stream);

/*
 * rlf_fused_lmhead_grpo under the objective variants of rlf_grpo_logp_loss_fwd_bwd_obj (same
 * formulas; the paper names GRPO / a PPO-style update in Sec. 2.3 and prints no objective):
 *   eps_clip_low, eps_clip_high   clip range (1 - eps_clip_low, 1 + eps_clip_high)
 *   aggregation   0: masked token mean (denom, if given, counts tokens);
 *                 1: mean over responses of each response's masked token mean (denom, if given,
 *                    counts responses); needs B <= T + 1
 *   skip_masked   1: rows with mask 0 are not multiplied at all, not even for their log-prob, which
 *                 reads NaN (with 46 % of the tokens inside tool observations, as in the Qwen3-4B
 *                 recipe, that is 46 % of the forward contraction); loss and gradients are unchanged.
 *                 0: every row's log-prob is produced.
 * Everything else (layouts, workspace, errors) as for rlf_fused_lmhead_grpo.
 */
rlf_status rlf_fused_lmhead_grpo_obj(const void *hidden, const void *W, int64_t T, int32_t D, int32_t V,
                                     const int32_t *ids, const int32_t *seq_id, const float *adv,
                                     int32_t B, const float *old_logp, const float *ref_logp,
                                     const uint8_t *mask, float eps_clip_low, float eps_clip_high,
                                     float beta_kl, int aggregation, int skip_masked,
                                     const int64_t *denom, float *logp_out, double *loss_out,
                                     void *grad_hidden, float *grad_W, int accumulate_grad_W,
                                     void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                     rlf_stream_t stream);

/*
 * Forward-only log-prob and entropy with the logits formed on the fly from the hidden states: the
 * pass that produces old_logp / ref_logp (the behaviour and reference policies of the PPO-style
 * update, paper Sec. 2.3.1; pi_theta of Sec. 2.2 is the language model's output head) without ever
 * writing [T, V] logits.
 *     z[t,:] = hidden[t,:] W^T;   logp[t] = z[t, ids[t]] - lse_t;   entropy[t] = lse_t - sum_v p_v z[t,v]
 *   hidden [T, D] bf16, W [V, D] bf16 (16-byte aligned; D a multiple of 64, V of 8);  ids [T] int32
 *   logp_out [T] fp32;  entropy_out [T] fp32 or NULL
 *   workspace  rlf_workspace_bytes(RLF_FN_FUSED_LOGP_ENTROPY, T, 0, 0, RLF_BF16) bytes, 256-byte aligned
 * An id outside [0, V) gives NaN log-prob (entropy is still produced) and RLF_DEV_BAD_TARGET; a
 * non-finite row gives NaN and RLF_DEV_NONFINITE.  Same contraction kernel, waits and tuning knobs as
 * rlf_fused_lmhead_grpo.  T = 0 is valid.
 */
rlf_status rlf_fused_lmhead_logp_entropy(const void *hidden, const void *W, int64_t T, int32_t D, int32_t V,
                                         const int32_t *ids, float *logp_out, float *entropy_out,
                                         void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                         rlf_stream_t stream);

/* Bytes of workspace the given entry point needs for these sizes (0 for unknown selectors). */
size_t rlf_workspace_bytes(int which_fn, int64_t T, int32_t V, int32_t D, rlf_dtype dt);

/*
 * One whole step from HOST buffers: copies the inputs to the device, runs
 * rlf_build_loss_mask -> rlf_group_advantage -> rlf_grpo_logp_loss_fwd_bwd,
 * copies loss (and, if asked, logp and mask) back and waits for the stream.
 * Host pointers should be page-locked for the copies to run at full rate.
 *
 *   h_*          host inputs, shapes as for the device entry points (contiguous groups of G)
 *   h_loss_out   [4] fp64 host;  h_logp_out [T] fp32 host or NULL;  h_mask_out [T] uint8 host or NULL
 *   d_arena      device scratch of rlf_step_arena_bytes(T, V, B, dt) bytes, 256-byte aligned; on
 *                return it holds grad_logits in place of the logits at offset 0 (row_stride = V)
 * Returns RLF_ERR_CUDA if a copy or the final wait fails; *h_dev_status (nullable) gets the device
 * status word.
 */
rlf_status rlf_grpo_step_host(const void *h_logits, rlf_dtype dt, int64_t T, int32_t V,
                              const int32_t *h_ids, const int32_t *h_cu_seqlens, int32_t B, int32_t G,
                              const float *h_rewards, const float *h_old_logp,
                              const float *h_ref_logp, int32_t open_id, int32_t close_id,
                              float adv_eps, float eps_clip, float beta_kl, double *h_loss_out,
                              float *h_logp_out, uint8_t *h_mask_out, int32_t *h_dev_status,
                              void *d_arena, size_t arena_bytes, rlf_stream_t stream);
size_t rlf_step_arena_bytes(int64_t T, int32_t V, int32_t B, rlf_dtype dt);

/* Launch shape of the fast logits kernel for later calls in this process: CTAs per cluster (1 to 16;
 * above 8 only with 256 threads and one_exp, for the plain token-mean training call), threads per CTA
 * (256, 512 or 1024), and whether each element's exponential is taken once
 * and kept as bf16 (one_exp = 1) or taken twice in fp32 (one_exp = 0; -1 = built-in choice).
 * cluster_ctas = 0 restores the built-in shape.  A shape that cannot hold a row in registers makes
 * rlf_grpo_logp_loss_fwd_bwd return RLF_ERR_UNSUPPORTED.  Results do not depend on the shape
 * beyond fp32 summation order (and, for one_exp, one extra bf16 rounding of the gradient). */
rlf_status rlf_tune_logits_kernel(int cluster_ctas, int threads_per_cta, int one_exp);

/* Grid sizing of the logits kernels for later calls in this process.  rows_per_cluster: a cluster of
 * the row kernels (training, skip-masked, row-per-cluster forward) handles about this many rows and
 * retires, so that several generations of clusters pass through the device during one launch (never
 * fewer clusters than fit at once); units_per_cta: the same for the CTAs of the streaming forward
 * pass, in row chunks.  0 restores the built-in choice (24 rows; 8 units).  Results do not depend
 * on either. */
rlf_status rlf_tune_logits_grid(int rows_per_cluster, int units_per_cta);

/* Form of the fused LM-head contractions for later calls in this process: 1 = pairs of CTAs share a
 * 256 x 256 tile (tcgen05 cta_group::2; the built-in choice), 0 = one CTA per 128 x 256 tile.
 * Results are identical up to fp32 summation order. */
rlf_status rlf_tune_lmhead(int pair_ctas);

/* Scheduling of the fused contractions for later calls in this process.  m_block: the persistent
 * CTAs (or CTA pairs) of the forward sweep that run at one time cover m_block row units (256 tokens
 * in pair form) times as many vocabulary splits as it takes to occupy them all; smaller blocks keep
 * less of the hidden states in L2 at a time and stream the head more often.  max_workers: upper
 * bound on the persistent CTAs (pairs) of every contraction launch.  chunk_tiles: 128-token tiles
 * per chunk of the backward (even; at most the 148 the workspace is sized for).  0 restores the
 * built-in choice (m_block = half the number of workers; one worker per SM or pair of SMs; 148
 * tiles).  Results do not depend on m_block or max_workers; the chunk size changes the order in
 * which grad_W is accumulated (fp32 rounding only). */
rlf_status rlf_tune_lmhead_schedule(int m_block, int max_workers, int chunk_tiles);

/* Backward scratch of the fused LM-head call for later calls in this process.  1 (the built-in choice):
 * the forward sweep stores exp(z - rho_t) against a per-row reference rho_t known before the sweep (the
 * row's fp32 target logit plus a constant), each row's factor c_t exp(rho_t - lse_t) is applied by the
 * gradient contractions, and there is no rescaling pass over the scratch; a chunk holding a row whose
 * reference proves unusable (its target's log-prob below about -78, or a non-finite sum) is redone the
 * other way, decided on the device.  0: exponentials against per-tile maxima, rescaled in place into
 * dZ by one more pass over the scratch.  Results agree to bf16 rounding of dZ.
 * two_accumulators (pair form only): 1 (built-in) = in the two gradient contractions a CTA pair
 * multiplies two 256-row tiles against each 256-column slab it stages (three quarters of the
 * shared-memory fill per flop, half the passes over the head or the hidden states); 0 = one tile per
 * pair with a double-buffered accumulator, as in the forward sweep.  Results are bit-identical. */
rlf_status rlf_tune_lmhead_backward(int row_reference, int two_accumulators);

/* Pacing of the fused contractions for later calls in this process.  1 (built-in): the persistent CTAs
 * (or pairs) of a contraction launch meet on a device counter before each of their work units, so
 * that workers which share operand slabs through L2 keep requesting them at about the same time;
 * without it they drift apart over a launch and each ends up streaming its operands from HBM by
 * itself.  Only loads are delayed, every wait is bounded, and a worker whose wait runs out goes on
 * unpaced.  0: no meeting points.  Results do not depend on it. */
rlf_status rlf_tune_lmhead_pacing(int on);

/* Number of kernels this library has launched in this process (for accounting). */
int64_t rlf_launch_count(void);

const char *rlf_status_string(rlf_status s);
int rlf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RLF_H_ */
