/* libjackpot: the OBRS token pass of Jackpot on one B200 (sm_100a).
 *
 * One pass over actor (rollout model, p_inf = q) and policy (p_target = p) logits
 * of shape [T, V].  Per token it computes both log-softmaxes and the sampled
 * token's log-probabilities, the two top-k sets, the OBRS acceptance probability
 * (Eq. obrs_accept), a Bernoulli accept/reject decision from a counter-based
 * generator, the top-k estimate of the normaliser Z (Section 4.4.1), the
 * batch-level bias correction kappa (Section 4.4.2) and the OBRS weights
 * (Algorithm 1, step 3).  A second call writes the gradient of the joint
 * objective (Eq. sys_joint_obj) with respect to both logit tensors.
 *
 * Conventions for every call
 *   - C linkage, plain pointers and sizes, no exceptions cross the boundary.
 *   - Unless a parameter says HOST, every data pointer is DEVICE memory on the
 *     context's device, owned by the caller, 16-byte aligned for logits and
 *     gradients.  The library never frees or keeps caller memory.
 *   - All work is enqueued on the context's stream; calls return after launch
 *     and never synchronise the device (the *_host variants do: they copy).
 *   - The context owns one workspace (per-token records), allocated with
 *     cudaMalloc on first use or by jp_reserve; it grows, never shrinks.
 *   - Return value: JP_OK or a negative jp_status; jp_last_error(ctx) gives a
 *     sentence.  Conditions found on the device (token id out of range,
 *     non-finite rows) never trap: such rows are counted in jp_stats and
 *     treated as masked, so the other rows' results do not depend on them.
 *   - A context is thread-compatible, not thread-safe.
 *   - Rows with mask[t] == 0 are not read; their outputs are accept = 0,
 *     weight = 0, logp = 0 and zero gradient rows.
 */
#ifndef JACKPOT_H_
#define JACKPOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct jp_ctx jp_ctx;

typedef enum {
  JP_OK = 0,
  JP_ERR_INVALID_ARG = -1,
  JP_ERR_ALIGNMENT = -2,
  JP_ERR_UNSUPPORTED = -3,
  JP_ERR_WORKSPACE = -4,
  JP_ERR_CUDA = -5,
  JP_ERR_TIMEOUT = -6,
  JP_ERR_STATE = -7,
  JP_ERR_TOO_LARGE = -8
} jp_status;

typedef enum { JP_BF16 = 0, JP_F32 = 1 } jp_dtype;
typedef enum { JP_LAMBDA_FIXED = 0, JP_LAMBDA_FROM_BUDGET = 1 } jp_lambda_mode;

enum { JP_MAX_TOPK = 128 };
enum { JP_STATIC_MAX_ROWS = 131072 };   /* row limit of jp_budget_lambda_static */
enum { JP_DESC_SPARSE_CAP = 2 };        /* jp_obrs_desc.flags, jp_obrs_forward_sparse_actor only: see there */
enum { JP_DESC_KL = 1 };                /* jp_obrs_desc.flags: also compute KL(p_target || p_inf) per row (one more
                                           pass over the rows) and report its batch mean in jp_stats.mean_kl_p_q */

/* Shapes, dtype, mode and optional outputs of one forward / backward call.
 * Zero-initialise, then set T, V and what differs from the defaults. */
typedef struct {
  int64_t T;             /* rows (token positions) in this call                          */
  int64_t V;             /* vocabulary size                                              */
  int64_t ld;            /* leading dimension of the logit (and gradient) rows in
                            elements; 0 means V.  ld * element size must be a multiple
                            of 16 bytes (for JP_F32 logits with a backward call: ld % 8 == 0) */
  int32_t dtype;         /* jp_dtype of the logits; gradients are always bf16            */
  int32_t lambda_mode;   /* jp_lambda_mode: meaning of lambda_or_budget                  */
  float c1;              /* clip on w_OBRS (Algorithm 1, step 3); <= 0 means no clip     */
  int32_t flags;         /* 0, or JP_DESC_KL                                             */
  int64_t token_offset;  /* global index of row 0: the accept draw of row t is keyed on
                            (seed, token_offset + t)                                     */
  /* Optional per-token outputs (device pointers, NULL to skip). */
  int32_t* topk_idx_actor;   /* [T,k] top-k(p_inf) indices, best first, ties by lower index */
  int32_t* topk_idx_policy;  /* [T,k] top-k(p_target)                                     */
  float* topk_val_actor;     /* [T,k] the actor logits at topk_idx_actor, as fp32         */
  float* topk_val_policy;    /* [T,k] the policy logits at topk_idx_policy                */
  float* accept_prob;        /* [T] a(x_t), Eq. obrs_accept                               */
  float* uniform;            /* [T] the uniform each decision compared against            */
  float* z_approx;           /* [T] Z_approx before the kappa correction (= Z when k >= V)*/
  float* z_exact;            /* [T] full-vocabulary Z (costs a second pass over the rows) */
  float* lse_actor;          /* [T] log sum_v exp(actor logit)                            */
  float* lse_policy;         /* [T]                                                       */
} jp_obrs_desc;

/* Batch statistics, written to DEVICE memory by the last kernel of a forward. */
typedef struct {
  int64_t n_valid;       /* N: rows with mask != 0, a token id inside [0, V) and usable numbers (see n_nonfinite) */
  int64_t n_accept;      /* accepted among them                                           */
  int64_t n_bad_token;   /* unmasked rows whose token id was outside [0, V): treated as masked */
  int64_t n_nonfinite;   /* unmasked rows with a NaN or +inf logit, or whose sampled token has probability 0
                            under the rollout model: treated as masked.  (log p_target(a_t) = -inf is a
                            legal row: the ratio is 0 and the token is rejected.)                       */
  double alpha_hat;      /* n_accept / n_valid (Section 4.4.2)                            */
  double mean_accept_prob; /* mean of a(x_t) over valid rows                              */
  double z_approx_mean;  /* mean of Z_approx over valid rows                              */
  double kappa;          /* alpha_hat / z_approx_mean; 1 if n_valid == 0 or the mean is 0 */
  double lambda_used;    /* the fixed lambda, or the one solved from the budget           */
  double mean_kl_p_q;    /* mean over valid rows of KL(p_target(.|s_t) || p_inf(.|s_t)), the actor-policy
                            divergence the paper tracks during training; NaN unless JP_DESC_KL was set
                            (in a chunked batch: on every chunk)                                     */
  int32_t status;        /* 0, or a jp_status raised on the device                        */
  int32_t pad;
} jp_stats;

/* Creates a context bound to `device` and to `cuda_stream` (a cudaStream_t cast
 * to void*, NULL = the default stream).  Allocates a few hundred bytes. */
jp_status jp_create(jp_ctx** out_ctx, int device, void* cuda_stream);
jp_status jp_destroy(jp_ctx* ctx);
/* Rebinds the stream later calls enqueue on. */
jp_status jp_set_stream(jp_ctx* ctx, void* cuda_stream);

/* Bytes of workspace that T_max rows with top-k size k need. */
size_t jp_obrs_workspace_bytes(int64_t T_max, int64_t V, int k);
/* Grows the workspace now (cudaMalloc) so that later calls allocate nothing. */
jp_status jp_reserve(jp_ctx* ctx, int64_t T_max, int64_t V, int k);

/* Forward pass over one [T,V] pair (Eq. obrs_accept, Eq. obrs_dist, Sections
 * 4.4.1-4.4.2, Algorithm 1 steps 2-3, Algorithm 2's accept test).
 *   actor_logits, policy_logits : [T, ld] of desc->dtype, each row read once
 *                                 (twice if desc->z_exact is set or k >= V)
 *   tokens  : [T] int32 sampled token ids a_t ~ p_inf
 *   mask    : [T] uint8, 0 = padding; NULL = all valid
 *   lambda_or_budget : lambda > 0 (JP_LAMBDA_FIXED) or the target mean acceptance
 *                      in (0,1] from which one batch-level lambda is solved
 *                      (Theorem 3.4 applied to the batch's sampled tokens)
 *   k       : 1..JP_MAX_TOPK selects the top-k estimate of Z; k >= V the exact
 *             sum over the vocabulary; JP_MAX_TOPK < k < V is JP_ERR_UNSUPPORTED
 *   seed    : key of the Philox4x32-10 stream of accept draws
 *   out_accept [T] uint8, out_weight [T] fp32 (min(kappa Z_approx max(lambda,
 *   p/q), c1) for every valid row, accepted or not), out_logp_actor /
 *   out_logp_policy [T] fp32 log-probabilities of the sampled token,
 *   out_stats : one jp_stats in device memory (may be NULL).
 * The per-token records stay in the context until the next forward or
 * jp_batch_begin; jp_obrs_backward reads them. */
jp_status jp_obrs_forward(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                          const void* policy_logits, const int32_t* tokens, const uint8_t* mask,
                          float lambda_or_budget, int k, uint64_t seed, uint8_t* out_accept,
                          float* out_weight, float* out_logp_actor, float* out_logp_policy,
                          jp_stats* out_stats);

/* Forward pass with the rollout model known only through what the rollout stored, as in the
 * paper's own pipeline (Algorithm 1, Phase 1: per token log p_inf(a_t) and TopK_inf(s_t), the
 * log-probabilities of its k_inf most likely tokens; Phase 2, step 2 builds V_k and Z_approx
 * from that record).  Only the policy tensor is streamed: half the bytes of jp_obrs_forward.
 *   policy_logits  : [T, ld] of desc->dtype (DEVICE), each row read once
 *   logp_inf_token : [T] fp32, log p_inf(a_t)
 *   topk_inf_idx   : [T, k_inf] int32 token ids of TopK_inf (any order; -1 = empty place)
 *   topk_inf_logp  : [T, k_inf] fp32 log p_inf of those tokens;  1 <= k_inf <= JP_MAX_TOPK
 *   k              : size of TopK_new, 1..JP_MAX_TOPK, k < V
 * Everything else as in jp_obrs_forward: log p_new(a_t) from the streamed row, acceptance
 * min(1, p_new(a_t) / (lambda p_inf(a_t))) (Eq. obrs_accept), lambda fixed or from a budget,
 * the accept draws, kappa and the weights (Section 4.4.2, Algorithm 1 step 3).
 * Z_approx = sum over V_k = TopK_inf U TopK_new of min(p_inf(x), p_new(x) / lambda).  For x in
 * TopK_new that the record does not hold, p_inf(x) is unknown and the paper does not say what to
 * take.  Default: the term is left out, so Z_approx stays a lower bound of Z, which the bias
 * correction of Section 4.4.2 assumes.  With JP_DESC_SPARSE_CAP in desc->flags it is bounded
 * instead: p_inf(x) <= the smallest stored probability, and all such terms together <= the
 * mass the record leaves; that is an upper bound of the dense path's Z_approx and may exceed Z.
 * out_z_lower / out_z_upper ([T] fp32, NULL to skip) give both.  With k_inf = V stored the two
 * coincide with jp_obrs_forward's exact mode.
 * Optional outputs of desc: topk_idx_policy, topk_val_policy, accept_prob, uniform, z_approx (the
 * reading in use), lse_policy; the actor-side ones and JP_DESC_KL are JP_ERR_UNSUPPORTED.  The
 * records this call leaves do not serve jp_obrs_backward (JP_ERR_STATE): the gradient with
 * respect to the rollout model's logits needs those logits. */
jp_status jp_obrs_forward_sparse_actor(jp_ctx* ctx, const jp_obrs_desc* desc, const void* policy_logits,
                                       const int32_t* tokens, const uint8_t* mask, const float* logp_inf_token,
                                       const int32_t* topk_inf_idx, const float* topk_inf_logp, int k_inf,
                                       float lambda_or_budget, int k, uint64_t seed, uint8_t* out_accept,
                                       float* out_weight, float* out_logp_policy, float* out_z_lower,
                                       float* out_z_upper, jp_stats* out_stats);

/* The row pass fused into the output layer, for one model (Section 4.4 names the
 * [tokens, vocabulary] logit tensor as the method's memory bottleneck; here it is never
 * written).  logits z[t, v] = sum_h hidden[t, h] * weight[v, h]: bf16 operands, fp32
 * accumulation on the tensor cores; the logits keep that fp32 value (they are not rounded to
 * bf16 as a stored logit tensor would be).  Per row t the call yields
 *   out_lse [T] fp32         log sum_v exp z[t, v]
 *   out_logp_token [T] fp32  z[t, tokens[t]] - lse
 *   out_topk_idx / out_topk_val [T, k]  the k largest logits, best first, equal values by lower
 *                            index, and their values; 1 <= k <= 64
 * which is what Algorithm 1 keeps of a forward pass (Phase 1: log p(a_t) and the top-k
 * log-probabilities; Phase 2 step 1 likewise for the policy).
 *   hidden : [T, ld_hidden] bf16, weight : [V, ld_weight] bf16 (the output layer's matrix, one row
 *            per vocabulary entry), both DEVICE, 16-byte aligned, pitches multiples of 16 bytes
 *            (ld = 0 means H); tokens [T] int32; mask [T] uint8 or NULL
 *   out_status : one int32 in DEVICE memory (may be NULL): 0, or JP_ERR_TIMEOUT if a wait inside
 *            the kernel ran out (results are then unspecified)
 * Rows with mask 0 or a token id outside [0, V) give lse = logp = 0 and indices -1.  Work is
 * enqueued on the context's stream; the context keeps a scratch buffer for partial results
 * (cudaMalloc on first use or growth). */
jp_status jp_lmhead_lse_topk(jp_ctx* ctx, const void* hidden, int64_t ld_hidden, const void* weight,
                             int64_t ld_weight, const int32_t* tokens, const uint8_t* mask, int64_t T,
                             int64_t H, int64_t V, int k, float* out_lse, float* out_logp_token,
                             int32_t* out_topk_idx, float* out_topk_val, int32_t* out_status);

/* The whole forward with both models' row passes fused into their output layers: neither
 * [T, V] logit tensor is ever stored (Section 4.4).  Each model's logits are
 * hidden[t, :] . weight[v, :] as in jp_lmhead_lse_topk (bf16 operands, fp32 accumulation, one
 * pass per model); for every entry of the two top-k lists the other model's logit is one more
 * dot product of a hidden state with a row of that model's output matrix; from there lambda
 * (fixed or from a budget), acceptance (Eq. obrs_accept), the accept draws, Z_approx over the
 * union of the two lists (Section 4.4.1), kappa and the weights (Section 4.4.2, Algorithm 1
 * step 3) run exactly as in jp_obrs_forward.
 *   desc : T, V (vocabulary), lambda_mode, c1, token_offset and the optional outputs are used;
 *          dtype and ld are ignored.  z_exact and JP_DESC_KL are JP_ERR_UNSUPPORTED (they need
 *          whole rows of logits).
 *   hidden_actor [T, ld_ha] / weight_actor [V, ld_wa] with hidden size H_actor, and the same for
 *   the policy (the two models may differ in hidden size): bf16, DEVICE, 16-byte aligned,
 *   pitches multiples of 16 bytes (ld = 0 means H).  1 <= k <= 64, k < V.
 * Outputs as in jp_obrs_forward.  The logits keep the precision of the fp32 accumulator, so
 * log-probs agree with a forward over stored bf16 logits only to the rounding of those.  The
 * records this call leaves do not serve jp_obrs_backward (JP_ERR_STATE). */
jp_status jp_obrs_forward_lmhead(jp_ctx* ctx, const jp_obrs_desc* desc, const void* hidden_actor, int64_t ld_ha,
                                 const void* weight_actor, int64_t ld_wa, int64_t H_actor,
                                 const void* hidden_policy, int64_t ld_hp, const void* weight_policy,
                                 int64_t ld_wp, int64_t H_policy, const int32_t* tokens, const uint8_t* mask,
                                 float lambda_or_budget, int k, uint64_t seed, uint8_t* out_accept,
                                 float* out_weight, float* out_logp_actor, float* out_logp_policy,
                                 jp_stats* out_stats);

/* Parameters of the backward pass (Eq. obrs_ppo, Eq. ppo_rollout, Eq.
 * distill_loss combined as Eq. sys_joint_obj; the PPO terms are maximised and
 * the distillation term minimised, so the loss is
 *   J = -L^{PPO-OBRS}(theta) - L^{PPO}(omega) + lambda_distill L^{distill}(omega),
 * a mean over the batch's N valid proposed tokens.  With the optional fields all
 * zero the loss is evaluated where the ratios r_theta = r_omega = 1 and F = 1 (the
 * first update after a rollout).  With them (Algorithm 1 steps 1, 3 and 4 for the
 * policy, Eq. ppo_rollout for the rollout model), per proposed token a_t:
 *   r_theta = p_new(a_t)/p_ref(a_t),  rho = weight_t * min(p_ref(a_t)/p_new(a_t), c2)
 *   policy term  Mask_t SG(rho) min(r_theta A_t, clip(r_theta, 1-eps_lo, 1+eps_hi) A_t)
 *   r_omega = p_omega(a_t)/p_omega_ref(a_t),  F = min(p_omega_ref(a_t)/p_inf(a_t), tis_cap)
 *   rollout term SG(F) min(r_omega A_t, clip(r_omega, 1-eps_lo, 1+eps_hi) A_t)
 * (weight_t is the forward's output and already carries the c1 clip; p_new(a_t) and
 * p_omega(a_t) are the forward's log-probs, kept in the context's records.)  A token
 * whose min sits on its clipped branch gets no gradient from that term. */
typedef struct {
  const float* advantages;  /* [T] A_t; NULL means 1                                   */
  float lambda_distill;     /* >= 0                                                    */
  float grad_out;           /* upstream scalar dL/dJ; 0 means 1                        */
  int64_t n_valid;          /* N of the whole batch; 0 = take it from the context's
                               last forward / jp_batch_finalize                        */
  int64_t record_offset;    /* index of row 0 in the context's records (the chunk's
                               token_offset for chunked batches, else 0)               */
  /* optional, device pointers, all may be NULL / 0 (see above) */
  const float* logp_ref;        /* [T] log p_ref(a_t), the policy before this update; NULL: r_theta = 1 */
  const float* logp_actor_ref;  /* [T] log p_omega,ref(a_t), the rollout model before this update
                                   (training engine); NULL: r_omega = 1                          */
  const float* logp_inf;        /* [T] log p_inf(a_t) as the rollout engine reported it; NULL: F = 1 */
  float eps_lo, eps_hi;         /* PPO clip range [1 - eps_lo, 1 + eps_hi]; both 0: no clipping   */
  float c2;                     /* cap on p_ref/p_new in rho; <= 0: none                          */
  float tis_cap;                /* cap of the truncated importance weight F; <= 0: none           */
  float* out_obj_policy;        /* [T] the policy term per token (0 for masked / rejected rows)   */
  float* out_obj_actor;         /* [T] the rollout term per token                                 */
  float* out_kl;                /* [T] KL(p_new(.|s_t) || p_omega(.|s_t)), the distillation term   */
  double* out_loss;             /* [4] J, L^{PPO-OBRS}, L^{PPO}, L^{distill}: this call's rows summed
                                   in a fixed order and divided by N (chunked batches: add the
                                   chunks' values); needs the three per-token outputs above       */
} jp_obrs_bwd_desc;

/* Writes dJ/d(actor logits) and dJ/d(policy logits), both [T, ld] bf16:
 *   d_policy[t,v] = -(g/N) accept_t w_t A_t (1[v = x_t] - p_t(v))
 *   d_actor[t,v]  = -(g/N) A_t (1[v = x_t] - q_t(v)) + (g lambda_distill/N)(q_t(v) - p_t(v))
 * (first-update form; in general w_t A_t becomes rho_t A_t r_theta on the live branch of
 * the min and 0 on the clipped one, and A_t becomes F_t A_t r_omega likewise).
 * accept / weight are the forward's outputs.  The log-sum-exps come from the
 * context's records of the matching forward (JP_ERR_STATE if there are none).
 * For bf16 logits d_actor_logits may alias actor_logits and d_policy_logits may
 * alias policy_logits (each element is read before it is overwritten). */
jp_status jp_obrs_backward(jp_ctx* ctx, const jp_obrs_desc* desc, const jp_obrs_bwd_desc* bwd,
                           const void* actor_logits, const void* policy_logits,
                           const int32_t* tokens, const uint8_t* mask, const uint8_t* accept,
                           const float* weight, void* d_actor_logits, void* d_policy_logits);

/* Chunked batches: kappa and a budget-derived lambda span the whole batch while
 * the logits exist one chunk at a time (Section 4.4.2: the calibration factor is
 * batch-wide).  begin -> chunk x n (rows stream once, records accumulate at
 * desc->token_offset .. +T) -> finalize (lambda, decisions, Z_approx, kappa,
 * weights for all T_total rows; outputs are [T_total]).  Rows no chunk covered
 * count as masked.  Exact mode (k >= V) needs a fixed lambda given at begin.
 * desc_outputs of jp_batch_finalize carries c1, the optional per-token outputs and
 * token_offset = the global row index of the batch's row 0 (0 unless this batch is
 * one shard of a larger one: the accept draws are keyed on the global index). */
jp_status jp_batch_begin(jp_ctx* ctx, int64_t T_total, int64_t V, int32_t dtype, int k,
                         float fixed_lambda_for_exact_mode);
jp_status jp_batch_chunk(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                         const void* policy_logits, const int32_t* tokens, const uint8_t* mask);
jp_status jp_batch_finalize(jp_ctx* ctx, const jp_obrs_desc* desc_outputs, float lambda_or_budget,
                            int32_t lambda_mode, uint64_t seed, uint8_t* out_accept,
                            float* out_weight, float* out_logp_actor, float* out_logp_policy,
                            jp_stats* out_stats);

/* Between the last jp_batch_chunk and jp_batch_finalize: the log-probs of the
 * sampled tokens that the streamed rows have left in the records, [T_total] fp32
 * each (0 for rows that are masked, have a bad token id or were not streamed), and
 * which rows are valid, [T_total] u8.  Any pointer may be NULL.  A batch spread over
 * several devices in budget mode gathers these from all of them, solves one lambda
 * over the whole batch (Theorem 3.4 applied to the batch's sampled tokens; see
 * jp_budget_lambda_static) and finalizes every shard with that fixed lambda: the
 * rows are still streamed once. */
jp_status jp_batch_logprobs(jp_ctx* ctx, float* out_logp_actor, float* out_logp_policy, uint8_t* out_valid);

/* A batch whose rows are spread over several devices (Section 4.4.2: the calibration
 * factor kappa is batch-wide).  Every device runs the forward on its shard, then
 *   jp_batch_totals       copies the shard's sums (N, accepted, sum of Z_approx, sum of
 *                         a(x_t)) to out_totals, [4] doubles in DEVICE memory;
 *   (the caller adds the shards' totals element-wise: one all-reduce of 32 bytes)
 *   jp_obrs_apply_totals  forms kappa = (accepted / N) / (sum of Z_approx / N) from the
 *                         summed totals (DEVICE, [4]; kappa = 1 if N = 0 or the sum is 0,
 *                         the rule of the one-device forward) and rewrites out_weight
 *                         [rows of the last forward / batch] = min(kappa Z_approx
 *                         max(lambda, p/q), c1) from the context's records (c1 <= 0: no
 *                         clip); out_stats (DEVICE, may be NULL) gets the batch-wide N,
 *                         accepted, alpha_hat, mean acceptance, mean Z_approx and kappa
 *                         beside this shard's own counters.
 * Both enqueue on the context's stream and do not wait.  JP_ERR_STATE without records.
 * jp_obrs_apply_kappa does the same with a kappa the caller already has. */
jp_status jp_batch_totals(jp_ctx* ctx, double* out_totals);
jp_status jp_obrs_apply_totals(jp_ctx* ctx, const double* totals, float c1, float* out_weight,
                               jp_stats* out_stats);
jp_status jp_obrs_apply_kappa(jp_ctx* ctx, double kappa, float c1, float* out_weight);

/* Vocabulary-parallel forward (Section 4.4 names the [tokens, vocabulary] logits as the
 * memory bottleneck; here every device holds a slice of the vocabulary's columns of both
 * tensors, as a vocabulary-parallel output layer leaves them).  Three steps per device:
 *
 *   jp_vshard_local   streams this device's columns once (the same row kernel as
 *                     jp_obrs_forward) and packs, per row, the slice's log-sum-exp of both
 *                     tensors, the sampled token's two logits if the slice holds it, and the
 *                     slice's two top-k lists with both logits of every entry, into
 *                     out_packed [T, jp_vshard_record_floats(k)] (device, 4-byte words);
 *   (the caller gathers every shard's out_packed into gathered [n_shards, T, words], shard
 *    order = ascending vocab_offset: an all-gather over the devices)
 *   jp_vshard_merge   turns the gathered lines into the records of the whole vocabulary:
 *                     lse = log sum_s exp(lse_s); log-probs of the sampled token from its
 *                     owner's logits; each top-k list = the k best of the shards' k best
 *                     under the same order (higher logit first, ties by lower index);
 *   jp_batch_finalize then completes the forward from the records exactly as for a chunked
 *                     batch: lambda (fixed or from a budget), acceptance (Eq. obrs_accept),
 *                     the accept draws, Z_approx (Eq. z_approx), kappa and the weights.
 *                     Every device ends with the same outputs for all T rows.
 *
 * desc describes the slice: T rows, V = the slice's width (> k), ld, dtype.  tokens are ids in
 * [0, V_total) (others make the row invalid and are counted in n_bad_token); vocab_offset is
 * the slice's first column.  The slices of the shards must tile [0, V_total) without overlap.
 * 1 <= k <= JP_MAX_TOPK (no exact mode: JP_ERR_UNSUPPORTED); n_shards <= 128, n_shards * k <= 4096
 * (JP_ERR_TOO_LARGE).  A row is valid if every shard found it valid.  All pointers device
 * memory owned by the caller; the calls enqueue on the context's stream and return.  The
 * context's records afterwards describe the whole vocabulary; the gradients of a slice come
 * from jp_vshard_backward.
 *
 * jp_vshard_backward: jp_obrs_backward for the columns [vocab_offset, vocab_offset + desc->V)
 * of rows whose records the merge and finalize left in this context.  The gradient of the
 * joint objective (Eq. sys_joint_obj) with respect to a logit needs, beside the logit itself,
 * only the row's two log-sum-exps and per-token scalars, all in the records, and the one-hot
 * term falls on the slice that holds the sampled token; so every device writes the gradient
 * of its own columns with no further exchange.  Arguments as for jp_obrs_backward with desc,
 * logits and gradients describing the slice and tokens holding ids in [0, V_total);
 * out_kl / out_loss need whole rows and are JP_ERR_UNSUPPORTED here.
 *
 * jp_vshard_local_push is jp_vshard_local with the all-gather folded into the export kernel:
 * gathered_of_shard is a HOST array of n_shards DEVICE pointers, entry p being shard p's gathered
 * buffer [n_shards, T, words] as this device can address it (its own buffer, and the peers'
 * through peer-mapped memory: CUDA IPC or symmetric memory, set up by the caller); the kernel
 * stores this shard's lines at [my_shard] of every one of them with plain global stores and
 * nothing else.  n_shards <= 16.  The caller makes sure every shard's push has completed
 * (its stream reached the end of the call, then a barrier over the devices) before any shard
 * runs jp_vshard_merge on its gathered buffer, and that no shard is still merging the previous
 * batch from a buffer that is pushed to again. */
size_t jp_vshard_record_floats(int k);
jp_status jp_vshard_local(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                          const void* policy_logits, const int32_t* tokens, const uint8_t* mask,
                          int64_t vocab_offset, int64_t V_total, int k, float* out_packed);
jp_status jp_vshard_local_push(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                               const void* policy_logits, const int32_t* tokens, const uint8_t* mask,
                               int64_t vocab_offset, int64_t V_total, int k, int n_shards, int my_shard,
                               float* const* gathered_of_shard);
jp_status jp_vshard_merge(jp_ctx* ctx, int n_shards, int my_shard, const float* gathered, int64_t T,
                          int64_t V_total, int k);
jp_status jp_vshard_backward(jp_ctx* ctx, const jp_obrs_desc* desc, const jp_obrs_bwd_desc* bwd,
                             const void* actor_logits, const void* policy_logits, const int32_t* tokens,
                             const uint8_t* mask, int64_t vocab_offset, const uint8_t* accept,
                             const float* weight, void* d_actor_logits, void* d_policy_logits);

/* Theorem 3.4 for single distributions: for every row t the lambda_t at which the
 * OBRS rule accepts exactly `budget` of the proposal's mass,
 *   sum_v min(q_t(v), p_t(v) / lambda_t) = budget,   q_t, p_t = softmax of the rows,
 * [T] fp32 (budget in (0, 1]; budget == 1 gives the smallest ratio p/q, the largest
 * lambda that still accepts everything).  Optionally KL(p_t || q_t), KL(p_t || q~_t)
 * with q~ the accepted distribution (Theorem 3.3: never larger; Figure 2b), and the
 * number of Newton steps taken, [T] each, NULL to skip.  Masked rows give 0.  Uses
 * desc's T, V, ld, dtype only; independent of the forward pass and its records.
 * This is the per-distribution budget of the theorem, not the batch-level lambda that
 * jp_obrs_forward solves in JP_LAMBDA_FROM_BUDGET mode. */
jp_status jp_obrs_row_lambda(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                             const void* policy_logits, const uint8_t* mask, float budget,
                             float* out_lambda, float* out_kl_before, float* out_kl_after,
                             int32_t* out_iterations);

/* Measurement aid (the paper has no counterpart): streams `bytes` of device memory
 * at src through a plain kernel `reps` times on the given stream and returns the
 * device time of one repetition in milliseconds.  dst == NULL: the buffer is only
 * read; else it is copied to dst (bytes more are written).  Pointers 16-byte aligned;
 * the call synchronises on the stream.  bench.py reports the read-only rate beside
 * the copy rate, since the forward pass only reads its logits. */
jp_status jp_probe_stream(const void* src, void* dst, int64_t bytes, int reps, void* cuda_stream,
                          float* out_ms_per_rep);

/* Same forward with every pointer in HOST memory (pinned memory makes the
 * copies asynchronous): the library stages the rows through device buffers it
 * owns, chunk by chunk with copies overlapping compute, writes the outputs back
 * and synchronises before returning.  chunk_rows = 0 picks a default.
 * Optional outputs of desc are not supported here and must be NULL. */
jp_status jp_obrs_forward_host(jp_ctx* ctx, const jp_obrs_desc* desc, const void* actor_logits,
                               const void* policy_logits, const int32_t* tokens,
                               const uint8_t* mask, float lambda_or_budget, int k, uint64_t seed,
                               uint8_t* out_accept, float* out_weight, float* out_logp_actor,
                               float* out_logp_policy, jp_stats* out_stats, int64_t chunk_rows);

/* The batch-level lambda for an acceptance budget, for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this entry point exists
 * for integration, not for the method.)
 *
 * Who this is for: code that runs where cudaMalloc is off limits.  Examples are a
 * training step whose device memory is entirely owned and budgeted by a framework
 * allocator, so that a hidden driver allocation could fail or fragment the pool; a
 * serving plug-in that may allocate only while it initialises; a latency-critical
 * loop, since cudaMalloc and cudaFree synchronise the device.  Every other entry
 * point of this library keeps its scratch in a context workspace that it grows
 * with cudaMalloc; this one calls no cudaMalloc, cudaFree or other allocating
 * routine.  Its scratch is a fixed array of about 1.7 MB inside the library's
 * device image, which every GPU that loads the library holds until the process
 * ends.
 *
 *   logp_actor, logp_policy : [T] fp32, DEVICE, log-probabilities of the sampled
 *                             tokens (outputs of jp_obrs_forward), read only
 *   mask    : [T] uint8 DEVICE, 0 = row takes no part; NULL = all rows
 *   T       : 0..JP_STATIC_MAX_ROWS; more rows return JP_ERR_TOO_LARGE and nothing
 *             is launched
 *   budget  : target mean acceptance in (0, 1]
 *   out_lambda : one fp32 in DEVICE memory; receives the lambda with
 *             (1/N) sum_t min(1, (p/q)(x_t) / lambda) = budget (1 if no row takes part)
 *   cuda_stream : cudaStream_t as void*, NULL = default stream; the work is
 *             enqueued on it on the CURRENT device and the call does not wait
 *
 * The first call on each device sets up: the driver loads the part of the library
 * image that holds the array (with lazy module loading this is when the device's
 * free memory drops by the array's size, once) and the array's device address is
 * looked up (a driver query).  Make that first call before any stream capture
 * begins.  Later calls change no allocation.
 * All calls on a device share the one array, which keeps whatever the previous
 * call left: each call rewrites what it reads, but two calls whose kernels overlap
 * on the GPU (different streams, no ordering between them) race on it.  Order
 * them, or use jp_obrs_forward with JP_LAMBDA_FROM_BUDGET, which has per-context
 * scratch.  Returns JP_OK, JP_ERR_INVALID_ARG, JP_ERR_TOO_LARGE or JP_ERR_CUDA. */
jp_status jp_budget_lambda_static(const float* logp_actor, const float* logp_policy,
                                  const uint8_t* mask, int64_t T, float budget, float* out_lambda,
                                  void* cuda_stream);

/* Self-test of the bounded waits (the paper has no counterpart).  Every wait inside the kernels
 * of this library (on a shared-memory barrier that the copy engine, another warp or the tensor
 * cores complete) gives up after a fixed number of SM clock cycles, sets JP_ERR_TIMEOUT in a
 * device status word and lets the kernel end instead of trapping or hanging.  This call runs
 * that routine against a barrier nobody completes, with a limit of limit_cycles (1 .. 2e9:
 * about a second at most): out_status (one int32, DEVICE) must read JP_ERR_TIMEOUT afterwards
 * and the context must work as before.  Enqueued on the context's stream; does not wait. */
jp_status jp_selftest_bounded_wait(jp_ctx* ctx, int64_t limit_cycles, int32_t* out_status);

const char* jp_status_string(jp_status s);
const char* jp_last_error(jp_ctx* ctx);
/* Number of kernel launches this context has enqueued so far. */
int64_t jp_launch_count(jp_ctx* ctx);
/* Per-launch device time of the row-stream kernel.  While timing is on, every
 * stream-kernel launch is bracketed by CUDA events on the context's stream (a
 * ring of 256 pairs).  jp_stream_kernel_times waits for the newest n of them,
 * writes their durations in milliseconds to out_ms (HOST memory, oldest first)
 * and returns how many it wrote.  Enabling or disabling restarts the count. */
jp_status jp_enable_kernel_timing(jp_ctx* ctx, int on);
int64_t jp_stream_kernel_times(jp_ctx* ctx, float* out_ms, int64_t n);

#ifdef __cplusplus
}
#endif
#endif /* JACKPOT_H_ */
