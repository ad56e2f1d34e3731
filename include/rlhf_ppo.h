/*
 * rlhf_ppo.h -- C ABI of the token-level PPO math for RLHF on NVIDIA B200 (sm_100a).
 *
 * The PPO stage of RLHF (paper, Section 2.1 "RLHF Training") runs four models: the actor, the
 * frozen reference that keeps the reward from diverging, the reward model that scores a whole
 * sequence, and the critic that estimates returns.  The actor generates responses; inference
 * passes of the four models turn them into experience; then the actor is trained to raise reward
 * while limiting its deviation from the old policy, and the critic is trained on the returns.
 * This library is the math between the models' outputs and their backward passes:
 *
 *   rlhf_gather_logprobs    log-prob of each generated token from a logits tensor (actor, reference)
 *   rlhf_kl_reward          per-token reward: KL penalty against the reference + sequence score
 *   rlhf_gae                advantages and returns from rewards and critic values
 *   rlhf_ppo_loss_fwd_bwd   clipped policy and value loss, gradient w.r.t. the logits and values
 *   rlhf_experience         the first three together (both log-prob passes in one kernel, reward + GAE in another)
 *   rlhf_whiten_advantages  optional masked whitening of the advantages between steps 3 and 4
 *   rlhf_ppo_stats          monitors of the policy step: approximate KL to the old policy, clip fraction
 *
 * The paper gives these quantities in prose only; the formulas are the standard definitions and
 * are written out beside each function.
 *
 * Conventions
 *  - B sequences, T response positions, V vocabulary entries.  lengths[b] in [0,T] is the number
 *    of valid response tokens of sequence b; positions t >= lengths[b] are padding.  Padded
 *    positions are ignored on input and every output is written as 0 there.
 *    N = sum_b lengths[b].
 *  - Every pointer is a DEVICE pointer owned by the caller unless it says "host".  The library
 *    allocates nothing, frees nothing and keeps no state between calls.  Calls are asynchronous
 *    on `stream` (a cudaStream_t passed as void*, NULL = the default stream) and never
 *    synchronise it (rlhf_poll_status excepted).
 *  - [B,T] arrays are fp32 (ids int64, lengths int32), row-major, T contiguous.
 *  - Logits are bf16 (binary16 through the *_ex entry points), addressed as base[b*stride_b + t*stride_t + v], strides in ELEMENTS,
 *    stride_t >= V.  For a full-sequence tensor [B,P+T,V] whose row P-1+t predicts response
 *    token t, pass base + (P-1)*V, stride_b = (P+T)*V, stride_t = V, and ids = input_ids + P with
 *    ids_stride_b = P+T.  Rows whose start address and byte length are multiples of 16 take the
 *    fast path; any other layout is handled by a slower kernel, not rejected.
 *  - A logit of -inf is a deleted vocabulary entry (probability 0, gradient 0).  It must not be
 *    the generated token's logit and a row must keep at least one finite logit; finite logits
 *    must satisfy |z| <= 1e38.  Violations produce NaN/inf in that row's outputs, never a fault.
 *  - Return value: an rlhf_status_t.  Errors the host can see (null pointers, sizes, strides,
 *    scalars out of range, workspace too small) are returned at once and nothing is launched.
 *    Errors only the device can see (an id outside [0,V), a length outside [0,T], a bounded wait
 *    that ran out) never fault; the code is OR-ed into the first word of the workspace, and
 *    rlhf_poll_status reports it.  A length outside [0,T] is clamped to that range.  A token
 *    whose id is outside [0,V) gets log-prob 0, policy-loss term 0 and an all-zero dlogits row;
 *    it still counts in N, and its value-loss term and dvalues entry (which do not depend on the
 *    id) are computed as for any valid token.
 *  - Arithmetic: fp32 throughout (exp/log of the softmax in base 2 with the hardware ex2); bf16
 *    outputs are rounded to nearest even.  Results do not depend on the order in which rows are
 *    scheduled: the loss is reduced in a fixed order, without floating-point atomics.
 */
#ifndef RLHF_PPO_H_
#define RLHF_PPO_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RLHF_OK = 0,
    RLHF_ERR_NULL = 1,          /* a required pointer is NULL */
    RLHF_ERR_SHAPE = 2,         /* B, T or V <= 0, or B*T above 2^29 */
    RLHF_ERR_ALIGN = 3,         /* a [B,T] array or the workspace is not aligned to its element / 256 B */
    RLHF_ERR_STRIDE = 4,        /* stride_t < V, negative stride, rows of different sequences overlap */
    RLHF_ERR_WORKSPACE = 5,     /* workspace smaller than rlhf_workspace_bytes(B,T) */
    RLHF_ERR_SCALAR = 6,        /* non-finite or out-of-range scalar argument */
    RLHF_ERR_CUDA = 7,          /* a CUDA runtime call or launch failed; see rlhf_last_cuda_error */
    RLHF_ERR_TOO_LARGE = 8,     /* rlhf_ppo_loss_fwd_bwd_noalloc: B*T above RLHF_NOALLOC_MAX_TOKENS */
    /* device-detected, sticky in the workspace, bit flags (may be OR-ed together) */
    RLHF_ERR_ID_RANGE = 16,     /* a generated-token id outside [0,V) at a valid position */
    RLHF_ERR_LENGTH_RANGE = 32, /* a length outside [0,T] (clamped) */
    RLHF_ERR_TIMEOUT = 64       /* an internal bounded wait ran out; outputs of this call are invalid */
} rlhf_status_t;

/* Element type of a logits tensor (and of the gradient written for it): the two 16-bit floating-point
 * types the paper's model families are run in (Section 3, "Workload and Setting").  The entry points
 * without a type argument take bf16; the *_ex ones take either.  Widening is exact; the gradient is
 * rounded to nearest even in the same type.  binary16 cannot hold magnitudes above 65504: a gradient
 * entry is at most |g| = grad_scale * |A| * rho / N in magnitude, so keep grad_scale such that this stays
 * below that bound (with grad_scale = 1 it always does), else the entry becomes +-inf. */
typedef enum {
    RLHF_BF16 = 0,
    RLHF_F16 = 1
} rlhf_dtype_t;

/* Human-readable name of a status (static storage; flags are joined with '|'). Host, never NULL. */
const char* rlhf_status_string(int status);

/* Text of the last CUDA runtime error this library saw on the calling thread ("" if none). */
const char* rlhf_last_cuda_error(void);

/* Host-side planning helper (no device access): which padded rows block `block` of a loss launch with
 * `n_blocks` persistent blocks zero-fills, for a batch with n_valid valid and n_padded padded tokens.
 * Valid rows are dealt round-robin (block i takes rows i, i+n_blocks, ...), so the first n_valid % n_blocks
 * blocks hold one valid row more than the others; a valid row moves twice the bytes of a padded one (read +
 * write against write only), so the other blocks first receive up to two padded rows each and the rest is
 * dealt evenly.  The share is the contiguous range [*start, *start + *count) of the row-major list of padded
 * tokens; the shares of blocks 0..n_blocks-1 tile [0, n_padded).  Returns RLHF_ERR_SHAPE for n_blocks <= 0,
 * a block outside [0, n_blocks) or negative counts, RLHF_ERR_NULL for NULL outputs.  The loss kernels use
 * the same rule on the device. */
int rlhf_pad_share(long long n_valid, long long n_padded, int n_blocks, int block,
                   long long* start, long long* count);

/* Bytes of scratch that rlhf_gather_logprobs, rlhf_experience and rlhf_ppo_loss_fwd_bwd need for a batch of B x T
 * tokens: O(B*T), never O(B*T*V) -- at most 16*B*T + 65536.  0 if B or T is not positive.
 * The workspace must be 256-byte aligned and must have been cleared once with rlhf_workspace_init
 * before its first use; it can then be reused by any number of calls on the same stream. */
size_t rlhf_workspace_bytes(int B, int T);

/* Zero the workspace (asynchronously, on `stream`). Needed once after allocation. */
int rlhf_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Synchronise `stream`, return the device-detected status flags accumulated in the workspace since
 * the last poll (RLHF_OK if none) and clear them. */
int rlhf_poll_status(void* workspace, void* stream);

/* Self-test of the library's failure detection (the paper has no counterpart).  Every kernel that waits on a
 * shared-memory barrier gives up after a bounded time, sets RLHF_ERR_TIMEOUT in the workspace and lets its block
 * drain instead of hanging.  This call launches one warp that waits, with that same code, on a barrier at which
 * nothing ever arrives, for at most limit_ns nanoseconds (0 < limit_ns <= 2e9), and returns.  Afterwards
 * rlhf_poll_status reports RLHF_ERR_TIMEOUT once, and the workspace is usable as before.  Nothing faults. */
int rlhf_selftest_bounded_wait(void* workspace, size_t workspace_bytes, unsigned long long limit_ns, void* stream);

/*
 * Step 1 -- log-probability of the generated tokens (Section 2.1: the actor and reference
 * inferences that produce the experience).  For t < lengths[b], with z = logits[b,t,:], y = ids[b,t]:
 *     out_logprobs[b,t] = z_y - log sum_v exp(z_v)
 * and 0 for t >= lengths[b].  One streaming read of each valid row; padded rows are not read.
 *   logits        bf16 [B,T,V] through (stride_b, stride_t)             read
 *   ids           int64, ids[b*ids_stride_b + t]                        read
 *   lengths       int32 [B]                                             read
 *   out_logprobs  fp32 [B,T]                                            written (all B*T entries)
 *   workspace     >= rlhf_workspace_bytes(B,T), 256-B aligned, initialised
 */
int rlhf_gather_logprobs(const void* logits, long long stride_b, long long stride_t,
                         const long long* ids, long long ids_stride_b, const int* lengths,
                         int B, int T, int V, float* out_logprobs,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * Step 1 with options: the element type of the logits (an rlhf_dtype_t) and, if out_entropy is not NULL, the
 * entropy of the softmax of every valid row,
 *     out_entropy[b,t] = - sum_v p_v log p_v,   p_v = exp(z_v - log sum_u exp(z_u))      (nats),
 * 0 at padded positions; a deleted entry (z_v = -inf) adds 0.  The entropy costs one more multiply-add per logit in
 * the same streaming pass, no extra memory traffic.  At a token whose id is out of range the log-prob is 0 (and
 * the status flag is set) but the entropy, which does not depend on the id, is still that of the row.
 * Everything else as rlhf_gather_logprobs.   RLHF_ERR_SCALAR for an unknown logits_dtype.
 */
int rlhf_gather_logprobs_ex(const void* logits, int logits_dtype, long long stride_b, long long stride_t,
                            const long long* ids, long long ids_stride_b, const int* lengths,
                            int B, int T, int V, float* out_logprobs, float* out_entropy,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Step 2 -- per-token reward (Section 2.1: the reference model prevents reward divergence, the
 * reward model gives the sequence-level score).  For t < lengths[b]:
 *     out_rewards[b,t] = -beta_kl * (lp_old[b,t] - lp_ref[b,t])
 *                        + [t == lengths[b]-1] * clamp(score[b], -reward_clip, +reward_clip)
 * and 0 for t >= lengths[b].  lp_old are the actor's log-probs when the experience was made.
 *   lp_old, lp_ref  fp32 [B,T]; score fp32 [B]; lengths int32 [B]      read
 *   out_rewards     fp32 [B,T]                                         written; may alias lp_old or lp_ref
 *   beta_kl >= 0, reward_clip >= 0 (use a huge value for "no clip"); both finite.
 */
int rlhf_kl_reward(const float* lp_old, const float* lp_ref, const float* score, const int* lengths,
                   int B, int T, float beta_kl, float reward_clip, float* out_rewards, void* stream);

/*
 * Step 3 -- generalised advantage estimation (Section 2.1: the critic estimates returns).
 * Backwards from the last valid token, with V_len = A_len = 0:
 *     delta_t = r_t + gamma * V_{t+1} - V_t
 *     A_t     = delta_t + gamma * lambda * A_{t+1}
 *     G_t     = A_t + V_t
 * out_adv = A, out_returns = G, both 0 for t >= lengths[b].
 *   rewards, values_old  fp32 [B,T]; lengths int32 [B]                  read
 *   out_adv, out_returns fp32 [B,T]                                     written; must not alias the inputs
 *   gamma, lambda in [0,1].
 */
int rlhf_gae(const float* rewards, const float* values_old, const int* lengths, int B, int T,
             float gamma, float lambda, float* out_adv, float* out_returns, void* stream);

/*
 * Optional, between steps 3 and 4 -- advantage whitening over the whole batch (Section 2.1 leaves the
 * normalisation of the advantages open; off unless the caller makes this call).  With N valid tokens,
 *     mean = (1/N) sum A,   var = (1/N) sum (A - mean)^2,   out_adv = (A - mean) / sqrt(var + eps)
 * at valid positions and 0 at padded ones; all zeros if N = 0 or var + eps = 0.  The sums are formed in
 * double precision in a fixed order (no floating-point atomics), so the result is bit-stable.
 *   adv       fp32 [B,T]; lengths int32 [B]                              read
 *   out_adv   fp32 [B,T]                                                 written; may be adv itself
 *   eps >= 0, finite.   workspace as for step 1.
 */
int rlhf_whiten_advantages(const float* adv, const int* lengths, int B, int T, float eps, float* out_adv,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Steps 1-3 together -- the whole experience phase (Section 2.1: the inferences of the actor,
 * reference, critic and reward models that turn generated responses into experience).  Computes
 * exactly what
 *     rlhf_gather_logprobs(actor) , rlhf_gather_logprobs(reference) , rlhf_kl_reward , rlhf_gae
 * compute when called in that order, with the same arithmetic (results are bit-identical to the four
 * calls), in two launches instead of four: one kernel streams both logits tensors, one small kernel
 * does the reward and the GAE scan of each sequence.
 *   actor_logits, ref_logits   bf16, each with its own strides, same ids / lengths               read
 *   score, values_old          as in steps 2 and 3                                                read
 *   lp_old                     fp32 [B,T] or NULL.  The log-probs of the KL term; NULL (the usual
 *                              case when the experience is being made) = the actor log-probs
 *                              computed by this call                                              read
 *   out_lp_actor, out_lp_ref, out_rewards, out_adv, out_returns   fp32 [B,T], distinct buffers    written
 *   workspace                  as for step 1
 * Scalars as in steps 2 and 3.
 */
int rlhf_experience(const void* actor_logits, long long actor_stride_b, long long actor_stride_t,
                    const void* ref_logits, long long ref_stride_b, long long ref_stride_t,
                    const long long* ids, long long ids_stride_b, const int* lengths,
                    const float* score, const float* values_old, const float* lp_old,
                    int B, int T, int V, float beta_kl, float reward_clip, float gamma, float lambda,
                    float* out_lp_actor, float* out_lp_ref, float* out_rewards, float* out_adv,
                    float* out_returns, void* workspace, size_t workspace_bytes, void* stream);

/* Steps 1-3 together with options: the element type of both logits tensors, and (if not NULL) the entropy of
 * the actor's rows as in rlhf_gather_logprobs_ex.  Everything else as rlhf_experience. */
int rlhf_experience_ex(const void* actor_logits, long long actor_stride_b, long long actor_stride_t,
                       const void* ref_logits, long long ref_stride_b, long long ref_stride_t, int logits_dtype,
                       const long long* ids, long long ids_stride_b, const int* lengths,
                       const float* score, const float* values_old, const float* lp_old,
                       int B, int T, int V, float beta_kl, float reward_clip, float gamma, float lambda,
                       float* out_lp_actor, float* out_lp_ref, float* out_rewards, float* out_adv,
                       float* out_returns, float* out_entropy, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Step 4 -- clipped PPO losses and their gradients (Section 2.1: the actor is trained to maximise
 * reward while limiting policy deviation, the critic is trained on the returns).  For each valid
 * token, with lp_new = z_y - lse(z) from the current logits (as step 1), rho = exp(lp_new - lp_old):
 *     l_pg = max(-A*rho, -A*clamp(rho, 1-clip_eps, 1+clip_eps))
 *     g    = grad_scale * (-A*rho) / N   if -A*rho >= -A*clamp(rho, ...)   else 0
 *     out_dlogits[b,t,v] = bf16( g * ([v == y] - exp(z_v - lse)) )
 *     vc   = values_old + clamp(values_new - values_old, -value_clip, +value_clip)
 *     l_vf = 1/2 * max((values_new - G)^2, (vc - G)^2)
 *     out_dvalues[b,t] = grad_scale * (values_new - G) / N   if (values_new-G)^2 >= (vc-G)^2   else 0
 *     *out_loss_pg = (1/N) sum l_pg        *out_loss_vf = (1/N) sum l_vf
 * Padded rows of out_dlogits are written as zeros, padded out_dvalues / out_lp_new as 0.  If N = 0
 * both losses and all gradients are 0.  Each valid row is read once from DRAM and written once.
 *   logits                       bf16 via (stride_b, stride_t)          read
 *   ids, lengths                 as step 1                              read
 *   lp_old, adv, values_new, values_old, returns   fp32 [B,T]           read
 *   out_loss_pg, out_loss_vf     fp32 scalars (device)                  written
 *   out_dlogits                  bf16 via (dl_stride_b, dl_stride_t)    written (all B*T rows); may be the
 *                                logits buffer itself with the same strides (in place), must not
 *                                otherwise overlap it
 *   out_dvalues                  fp32 [B,T]                             written
 *   out_lp_new                   fp32 [B,T] or NULL                     written if given
 *   clip_eps in (0,1), value_clip >= 0, grad_scale finite.
 */
int rlhf_ppo_loss_fwd_bwd(const void* logits, long long stride_b, long long stride_t,
                          const long long* ids, long long ids_stride_b, const int* lengths,
                          const float* lp_old, const float* adv, const float* values_new,
                          const float* values_old, const float* returns,
                          int B, int T, int V, float clip_eps, float value_clip, float grad_scale,
                          float* out_loss_pg, float* out_loss_vf,
                          void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                          float* out_dvalues, float* out_lp_new,
                          void* workspace, size_t workspace_bytes, void* stream);

/* Step 4 with the element type of logits and out_dlogits (an rlhf_dtype_t; both tensors have the same type).
 * Everything else as rlhf_ppo_loss_fwd_bwd.  RLHF_ERR_SCALAR for an unknown logits_dtype. */
int rlhf_ppo_loss_fwd_bwd_ex(const void* logits, int logits_dtype, long long stride_b, long long stride_t,
                             const long long* ids, long long ids_stride_b, const int* lengths,
                             const float* lp_old, const float* adv, const float* values_new,
                             const float* values_old, const float* returns,
                             int B, int T, int V, float clip_eps, float value_clip, float grad_scale,
                             float* out_loss_pg, float* out_loss_vf,
                             void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                             float* out_dvalues, float* out_lp_new,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Monitors of the policy step (Section 2.1: the actor is trained "while minimizing policy deviation"; these two
 * numbers are how that deviation is watched).  From the log-probs that step 4 returns in out_lp_new:
 *     rho = exp(lp_new - lp_old)
 *     out_stats[0] = approx_kl = (1/N) sum ((rho - 1) - log rho)          (non-negative, 0 on policy)
 *     out_stats[1] = clip_frac = (1/N) #{ -A*clamp(rho, 1-clip_eps, 1+clip_eps) > -A*rho }
 * over the valid tokens; both 0 if N = 0.  clip_frac is the share of tokens to which step 4 gives a zero
 * gradient; a token whose ratio sits on the edge of the interval to within float32 rounding may be counted on
 * either side.  Sums in double precision in a fixed order.
 *   lp_new, lp_old, adv   fp32 [B,T]; lengths int32 [B]                 read
 *   out_stats             fp32 [2] (device)                              written
 *   clip_eps in (0,1).   workspace as for step 1.
 */
int rlhf_ppo_stats(const float* lp_new, const float* lp_old, const float* adv, const int* lengths, int B, int T,
                   float clip_eps, float* out_stats, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Step 4 for callers that cannot provide a workspace.  (The paper has no counterpart to this
 * entry point; it exists for integration reasons only.)
 *
 * Some callers have no way to obtain scratch memory: a plug-in that is handed raw tensor pointers
 * but no allocator; a process in which a framework's caching allocator has already reserved the
 * whole device, so that a direct cudaMalloc fails; a latency-critical loop that must not take the
 * implicit device synchronisation of cudaMalloc/cudaFree.  For them this variant computes exactly
 * what rlhf_ppo_loss_fwd_bwd computes, with the same arguments minus the workspace, and takes
 * its scratch from a fixed array that is part of the library image in device memory.
 *
 *  - The array holds the scratch for at most RLHF_NOALLOC_MAX_TOKENS = 65536 tokens (B*T); it is
 *    about 280 KB and is resident on every GPU that loads the library, until the process exits.
 *    A larger batch is refused with RLHF_ERR_TOO_LARGE and nothing is launched.
 *  - The call allocates and frees nothing, directly or through any library.
 *  - The first call on each device looks up the device address of the array (with that device
 *    current) and remembers it.  Make that first call outside any stream capture.  The remembered
 *    address does not survive a cudaDeviceReset in the same process.
 *  - All calls on one device share the array, and it keeps what the previous call left in it.
 *    The call itself clears the words that must start at zero.  Two calls whose kernels can run
 *    at the same time on one device (different streams without an ordering between them) race on
 *    the array and give undefined results: keep calls on one stream, or order them with events.
 *  - out_device_status: optional device pointer to one 32-bit word; if given, the device-detected
 *    status flags of this call (RLHF_ERR_ID_RANGE, ...; 0 if none) are copied there on `stream`.
 *  Everything else (arguments, layouts, aliasing rules, return value) is as for
 *  rlhf_ppo_loss_fwd_bwd.
 */
#define RLHF_NOALLOC_MAX_TOKENS 65536

int rlhf_ppo_loss_fwd_bwd_noalloc(const void* logits, long long stride_b, long long stride_t,
                                  const long long* ids, long long ids_stride_b, const int* lengths,
                                  const float* lp_old, const float* adv, const float* values_new,
                                  const float* values_old, const float* returns,
                                  int B, int T, int V, float clip_eps, float value_clip, float grad_scale,
                                  float* out_loss_pg, float* out_loss_vf,
                                  void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                                  float* out_dvalues, float* out_lp_new,
                                  unsigned int* out_device_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RLHF_PPO_H_ */
