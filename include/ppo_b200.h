/*
 * ppo_b200.h -- C ABI of the per-token PPO-for-RLHF hot path (arXiv 2403.17031) for NVIDIA
 * B200 (sm_100a).
 *
 * The path, in the order a PPO iteration runs it:
 *   1. ppo_logprob_entropy      log-prob of each sampled response token and entropy of the
 *                               temperature-scaled distribution, for the policy and again for
 *                               the frozen SFT reference
 *   2. ppo_truncate_and_score   the "EOS trick": cut at the first EOS, fill [PAD], -1 score
 *   3. ppo_kl_rewards           per-token KL penalty, reward-model score on the last token
 *   4. ppo_gae                  reverse-time generalised advantage estimation
 *   5. ppo_whiten               masked mean/variance normalisation of the advantages
 *   6. ppo_loss_fwd_bwd         clipped policy loss + clipped value loss and their gradients
 *   7. ppo_lmhead_logprob_entropy  step 1 with the LM-head GEMM fused in (logits never stored)
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless a comment says "host".
 *     The library allocates nothing; scratch lives in a caller-provided workspace.
 *   - Work is enqueued on the caller's stream (`stream` is a cudaStream_t passed as void*;
 *     NULL is the default stream) and the call returns without synchronising, except
 *     ppo_last_device_status and the *_host entry points.
 *   - Return value: 0 on success; a negative PPO_ERR_* code for an argument error found on
 *     the host before anything is launched; a positive value is a cudaError_t reported by
 *     the CUDA runtime.  Nothing traps, aborts or falls back to a CPU path.
 *   - Outputs are completely overwritten (positions with mask 0 receive 0); inputs are never
 *     modified; outputs must not alias inputs unless stated.
 *   - Data-dependent soft errors (a token id outside [0,V), an all-zero mask, a bounded wait
 *     that ran out) set bits in a status word inside the workspace; the affected outputs are
 *     NaN.  Read it with ppo_last_device_status.
 *   - Logits: row-major [rows, V], dtype PPO_F32 or PPO_BF16.  The fast kernels need the base
 *     address and the row pitch to be multiples of 16 bytes and V a multiple of 16/sizeof(elt);
 *     anything else takes a slower element-wise kernel with the same results.
 */
#ifndef PPO_B200_H
#define PPO_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* logits storage types */
#define PPO_F32 0
#define PPO_BF16 1

/* host-side argument errors (returned, never thrown) */
#define PPO_OK 0
#define PPO_ERR_NULL (-1)        /* a required pointer is NULL */
#define PPO_ERR_SHAPE (-2)       /* a size is <= 0, too large, or inconsistent */
#define PPO_ERR_PARAM (-3)       /* temperature <= 0, negative clip range, eos_id == pad_id, non-finite */
#define PPO_ERR_ALIGN (-4)       /* pointer alignment below the element size / documented minimum */
#define PPO_ERR_DTYPE (-5)       /* unknown dtype code */
#define PPO_ERR_UNSUPPORTED (-6) /* shape outside what the kernel handles (documented per call) */

/* bits of the device status word */
#define PPO_DEV_BAD_TOKEN 1      /* a token id was outside [0, V): that row's outputs are NaN */
#define PPO_DEV_EMPTY_MASK 2     /* mask selected no element: statistics / losses are 0 */
#define PPO_DEV_TIMEOUT 4        /* a bounded wait inside a kernel gave up; outputs are invalid */
#define PPO_DEV_BAD_ROW 8        /* ppo_sample_logprob_entropy: a row had a NaN / +inf or no finite logit: token -1 */
#define PPO_DEV_BAD_REUSE 16     /* ppo_loss_fwd_bwd_next_epoch: the workspace does not hold this mask's row order; nothing was written */

/* indices into the losses[8] output of ppo_loss_fwd_bwd */
enum { PPO_LOSS_PG = 0, PPO_LOSS_VF = 1, PPO_LOSS_TOTAL = 2, PPO_LOSS_APPROX_KL = 3,
       PPO_LOSS_PG_CLIPFRAC = 4, PPO_LOSS_VF_CLIPFRAC = 5, PPO_LOSS_ENTROPY = 6, PPO_LOSS_N = 7 };

/*
 * Hyper-parameters of the path.  Defaults (ppo_default_params) are the paper's Table "PPO
 * hyperparameters": temperature 0.7, kl_coef (beta) 0.05, gamma 1.0, lam 0.95, cliprange
 * (epsilon) 0.2, cliprange_value (epsilon-hat) 0.2, vf_coef (c1) 0.1; no_eos_score -1 from the
 * "EOS trick"; whiten_eps 1e-8 from the whiten() listing; eos_id 0 (Pythia <|endoftext|>);
 * pad_id must be set by the caller to a [PAD] id different from eos_id (section "Dataset ->
 * ... do not use EOS synonymously as [PAD]"); the default 1 is only a placeholder.
 * whiten_rewards (default 0 = off): detail "(Optional) Reward whitening" - when non-zero, ppo_step
 * whitens the per-token rewards of the batch over its real tokens with shift_mean = 0 (mean kept)
 * before GAE; callers of the separate entry points do the same with ppo_whiten between
 * ppo_kl_rewards and ppo_gae.  Only ppo_step reads this field.
 */
typedef struct ppo_params {
    float temperature, kl_coef, gamma, lam, cliprange, cliprange_value, vf_coef, no_eos_score,
        whiten_eps;
    int32_t eos_id, pad_id;
    int32_t whiten_rewards;
} ppo_params;

void ppo_default_params(ppo_params *p /* host */);

/* Library version: major * 10000 + minor * 100 + patch. */
int ppo_version(void);

/*
 * Process-wide tuning switches; every setting computes the same results.  Returns 0, or
 * PPO_ERR_PARAM for an unknown key/value.  Not thread-safe against concurrent launches.
 *   PPO_OPT_LOSS_ROW_CACHE  how ppo_loss_fwd_bwd keeps a row between its statistics pass and its
 *                           gradient pass: 0 = choose by row size (default), 1 = in shared memory
 *                           whenever the row fits one block, 2 = re-read it from global memory/L2
 *                           (applies to the direct-load kernels only)
 *   PPO_OPT_ROW_ENGINE      which kernels stream the logits: 0 = default (the loss through the
 *                           bulk-copy row engine when the shape allows, log-prob/entropy through
 *                           direct loads), 1 = direct loads for both, 2 = row engine for both
 */
#define PPO_OPT_LOSS_ROW_CACHE 1
#define PPO_OPT_ROW_ENGINE 2
int ppo_set_option(int key, int value);

/*
 * Workspace.  ppo_workspace_bytes gives the size (a multiple of 256) that serves every call
 * below for batches up to B x T tokens (V is accepted for future use); the fused LM-head call
 * needs ppo_lmhead_workspace_bytes(M, K, V) instead (use the larger of the two to share one
 * buffer).  The buffer must be 256-byte aligned and must be cleared once with
 * ppo_workspace_init before its first use.  One workspace serves one stream at a time.
 */
size_t ppo_workspace_bytes(int32_t B, int32_t T, int64_t V);
size_t ppo_lmhead_workspace_bytes(int64_t M, int64_t K, int64_t V);
int ppo_workspace_init(void *workspace, size_t bytes, void *stream);

/*
 * Waits for `stream`, copies the status word to *status (host), clears it on the device, and
 * returns 0 (or a CUDA error).  The word accumulates PPO_DEV_* bits from every call that was
 * given this workspace since the last read.
 */
int ppo_last_device_status(void *workspace, void *stream, int *status /* host */);

/*
 * Step 1.  For every row r of logits [rows, V] (row pitch `row_stride` elements):
 *     z = logits[r, :] / temperature,   lse = log sum_j exp(z_j),
 *     logprob[r] = z[tokens[r]] - lse,  entropy[r] = -sum_j softmax(z)_j * log softmax(z)_j.
 * The paper fixes the temperature (Table "PPO hyperparameters": 0.7) and requires policy and
 * SFT reference to be scored identically (Eq. "RL"; section "Disable dropout ...": ratios
 * are 1 in the first epoch); call once per model.  Row [b,t] must be the distribution that
 * response token t was sampled from (the caller has already shifted/sliced the sequence
 * logits).  -inf logits are allowed and carry zero probability.
 *   mask     nullable [rows] u8: rows with 0 are not read and output 0.
 *   entropy, lse   nullable [rows] f32.
 *   workspace      nullable; without it out-of-range tokens still give NaN but set no status.
 * Errors: PPO_ERR_NULL, PPO_ERR_SHAPE (rows < 0, V <= 0, row_stride < V, V >= 2^31),
 * PPO_ERR_PARAM (temperature), PPO_ERR_DTYPE, PPO_ERR_ALIGN (base not element-aligned).
 * rows == 0 is a successful no-op.
 */
int ppo_logprob_entropy(const void *logits, int dtype, int64_t rows, int64_t V, int64_t row_stride,
                        const int32_t *tokens, const uint8_t *mask, float temperature,
                        float *logprob, float *entropy, float *lse, void *workspace, void *stream);

/*
 * Step 2, the "EOS trick" (section "PPO Training -> EOS trick"): responses always have T
 * sampled tokens; the response is cut at its first eos_id, later positions become pad_id, and
 * a response without EOS has its score REPLACED by no_eos_score (-1).  The EOS token itself
 * stays a real token (the reward model's score is read on it).
 *   responses      [B,T] i32 in;  scores [B] f32 in (nullable together with scores_out)
 *   responses_out  [B,T] i32 (nullable; may alias responses)
 *   eos_index      [B] i32, -1 when absent (nullable)
 *   seq_len        [B] i32 = eos_index+1, or T (nullable)
 *   mask           [B,T] u8 = (t < seq_len) (nullable)
 *   scores_out     [B] f32 (nullable)
 * Integer outputs are exact.  Errors: PPO_ERR_NULL, PPO_ERR_SHAPE, PPO_ERR_PARAM (eos_id ==
 * pad_id).
 */
int ppo_truncate_and_score(const int32_t *responses, int32_t B, int32_t T, int32_t eos_id,
                           int32_t pad_id, const float *scores, float no_eos_score,
                           int32_t *responses_out, int32_t *eos_index, int32_t *seq_len,
                           uint8_t *mask, float *scores_out, void *stream);

/*
 * Step 3 (Eq. "RL": R = r_phi - beta * KL[pi_theta || pi_SFT]; figure "reward vs value": the
 * reward vector holds a KL penalty per token and the reward-model score on the EOS token):
 *     kl[b,t] = mask * (logprob - ref_logprob)         (the k1 estimator at the sampled token)
 *     rewards[b,t] = -kl_coef * kl[b,t];  rewards[b, seq_len[b]-1] += scores[b]
 * All arrays [B,T] f32 except seq_len [B] i32, scores [B] f32 (already passed through step 2).
 * kl and rewards are nullable (at least one required).
 */
int ppo_kl_rewards(const float *logprob, const float *ref_logprob, const uint8_t *mask,
                   const int32_t *seq_len, const float *scores, int32_t B, int32_t T,
                   float kl_coef, float *kl, float *rewards, void *stream);

/*
 * The three curves of the paper's figure of PPO learning curves, from the outputs of steps 2 and 3:
 *     out3[0] = mean over b of R_b,  R_b = scores[b] - kl_coef * sum_t kl[b,t]   (Eq. "RL" with the
 *               KL of a response estimated by its summed per-token k1 terms)
 *     out3[1] = mean over b of sum_t kl[b,t]   (the figure's KL curve: per-token KL terms between RL
 *               and SFT policy summed per response, then averaged over the responses)
 *     out3[2] = mean over b of scores[b]       (pass step 2's scores_out for what PPO optimises)
 * kl [B,T] f32 (step 3), scores [B] f32, out3 [3] f32, all device.  mask [B,T] u8 is nullable: with
 * it, positions with mask 0 are left out of the sums; without it every position counts (step 3
 * already writes 0 behind the responses).  Means are over the B responses.  One block, fp64 sums in
 * a fixed order.  B, T >= 1; errors: PPO_ERR_SHAPE, PPO_ERR_NULL, PPO_ERR_PARAM (kl_coef not finite).
 */
int ppo_rollout_curves(const float *kl, const uint8_t *mask, const float *scores, int32_t B, int32_t T,
                       float kl_coef, float *out3, void *stream);

/*
 * Step 4, GAE with the table's gamma and lambda.  The episode ends after the last real token
 * (the value function predicts the end-of-episode return, section "Value model initializes
 * from the reward model"), so nothing is bootstrapped beyond seq_len-1:
 *     delta_t = r_t + gamma * V_{t+1} - V_t,   A_t = delta_t + gamma * lam * A_{t+1},
 *     returns_t = A_t + V_t;   V_t = A_t = 0 for t >= seq_len;  zeros are written there.
 * One warp per sequence runs a segmented reverse scan of affine maps in fp64 and rounds once.
 * Any T >= 1 is supported.
 */
int ppo_gae(const float *rewards, const float *values, const int32_t *seq_len, int32_t B, int32_t T,
            float gamma, float lam, float *advantages, float *returns, void *stream);

/*
 * Step 5, the paper's whiten() (listing in section "Reward whitening"; applied to advantages
 * in section "Advantage whitening") over the entries with mask 1 of one flat array:
 *     mean = sum(m*x)/n,  var = sum(m*(x-mean)^2)/n  (biased),
 *     out = (x - mean) * rsqrt(var + eps);  if (!shift_mean) out += mean;  out = 0 where m == 0.
 * shift_mean != 0 (the listing's default, used for advantages) leaves zero mean.
 *   mask nullable (all ones); out may alias x; stats3 nullable [3] f32 = {mean, var, n}.
 * One thread block computes the statistics in fp64 in a fixed order (bit-reproducible).
 * n == 0 writes zeros and sets PPO_DEV_EMPTY_MASK (when a workspace is given).
 */
int ppo_whiten(const float *x, const uint8_t *mask, int64_t n_elems, int shift_mean, float eps,
               float *out, float *stats3, void *workspace, void *stream);

/*
 * Step 6.  With lp_new computed from `logits` as in step 1 (temperature from *p),
 * rho = exp(lp_new - old_logprob), A = advantages, v = values_new:
 *     pg = max(-A*rho, -A*clip(rho, 1-cliprange, 1+cliprange))
 *     vc = clip(v, values_old - cliprange_value, values_old + cliprange_value)
 *     vf = max((v - returns)^2, (vc - returns)^2)
 *     losses[PG] = sum(m*pg)/n,  losses[VF] = 0.5*sum(m*vf)/n,  losses[TOTAL] = PG + vf_coef*VF
 * (Table "PPO hyperparameters": cliprange 0.2, cliprange_value 0.2, vf_coef 0.1, value-loss
 * clipping on, one minibatch so n counts the whole call's real tokens), and the gradients of
 * losses[TOTAL]:
 *     dlogits[b,t,j] = g * (1[j == token] - softmax(z)_j) / temperature,
 *         g = (m/n) * (-A*rho) unless the clipped branch is strictly larger (then 0)
 *     dvalues[b,t]   = vf_coef * (m/n) * (v - returns) unless the clipped branch is strictly larger
 * Also losses[APPROX_KL] = 0.5*mean((lp_new-old_logprob)^2), the two clip fractions, the mean
 * entropy and n.  Rows with mask 0 are not read; their dlogits rows are zero-filled.
 *   logits   [B,T,V] contiguous (pitch V);   dlogits same shape and dtype (nullable: forward
 *            statistics and dlogprob only);  must not alias logits
 *   tokens, mask(u8), old_logprob, advantages, values_new, values_old, returns: [B,T]
 *   losses   [8] f32;  dvalues [B,T] f32;  new_logprob, entropy, dlogprob: nullable [B,T] f32
 *   workspace required (ppo_workspace_bytes(B,T,V)).
 * Per-row partial sums are reduced in a fixed order in fp64, so results are bit-reproducible.
 */
int ppo_loss_fwd_bwd(const void *logits, int dtype, int32_t B, int32_t T, int64_t V,
                     const int32_t *tokens, const uint8_t *mask, const float *old_logprob,
                     const float *advantages, const float *values_new, const float *values_old,
                     const float *returns, const ppo_params *p /* host */, float *losses,
                     void *dlogits, float *dvalues, float *new_logprob, float *entropy,
                     float *dlogprob, void *workspace, void *stream);

/*
 * The same call for the later PPO epochs of a batch (the paper's table: 4 epochs per batch): it must follow a
 * ppo_loss_fwd_bwd, ppo_loss_fwd_bwd_next_epoch or ppo_step call on the same workspace with the same mask
 * pointer, B and T, with no other call that uses this workspace in between.  The token count and row order
 * that call left in the workspace are reused, which saves the prologue launch; all other arguments (logits,
 * old_logprob, ...) may differ, the results are those of ppo_loss_fwd_bwd.  The kernel checks that the
 * order in the workspace was built from this mask pointer, row count and workspace; if not, it sets
 * PPO_DEV_BAD_REUSE in the device status and writes nothing.  The CONTENT of mask must not have changed
 * since (not checked).
 */
int ppo_loss_fwd_bwd_next_epoch(const void *logits, int dtype, int32_t B, int32_t T, int64_t V,
                     const int32_t *tokens, const uint8_t *mask, const float *old_logprob,
                     const float *advantages, const float *values_new, const float *values_old,
                     const float *returns, const ppo_params *p /* host */, float *losses,
                     void *dlogits, float *dvalues, float *new_logprob, float *entropy,
                     float *dlogprob, void *workspace, void *stream);

/*
 * Step 6 when the logits were never materialised (fused LM head): same losses and dvalues from
 * a given new_logprob [B,T]; dlogprob [B,T] receives g.  entropy nullable [B,T] (averaged into
 * losses[ENTROPY] when given, else 0).
 */
int ppo_loss_from_logprob(const float *new_logprob, const float *entropy, int32_t B, int32_t T,
                          const uint8_t *mask, const float *old_logprob, const float *advantages,
                          const float *values_new, const float *values_old, const float *returns,
                          const ppo_params *p /* host */, float *losses, float *dlogprob,
                          float *dvalues, void *workspace, void *stream);

/*
 * Step 1 for the policy and the frozen reference in ONE launch (same tokens, same shape, row pitch V):
 * logprob / entropy (nullable) from policy_logits, ref_logprob from ref_logits; otherwise exactly
 * ppo_logprob_entropy called twice (which is what happens for layouts without 16-byte packs).  One
 * launch boundary less, at which the SMs would drain and refill; with a mask, rows with mask 0 are
 * skipped in both tensors (outputs 0).
 */
int ppo_logprob_entropy_pair(const void *policy_logits, const void *ref_logits, int dtype, int64_t rows, int64_t V,
                             const int32_t *tokens, const uint8_t *mask, float temperature, float *logprob,
                             float *entropy, float *ref_logprob, void *workspace, void *stream);

/*
 * Temperature sampling fused with step 1 (Table "PPO hyperparameters": temperature): draws one token
 * per row from softmax(logits / temperature) and returns its log-prob, the row's entropy and
 * log-sum-exp from the same single pass over HBM.  The draw is reproducible and defined as follows:
 *   uniform(w) = (floor(w / 2^9) + 1/2) * 2^-23 for a 32-bit word w    (an fp32 number in (0, 1))
 *   words come from Philox4x32-10 with key = seed; y_j = logit_j * log2(e) / temperature
 *   The row is dealt into 256 classes in runs of 8 elements, class(j) = (j / 8) mod 256, and an exponential
 *   race (the Gumbel-max rule) is run in two levels:
 *   level 1:  W_c = sum of 2^(y_j) over class c;  v_c = uniform(word c % 4 of counter (2^31 + c / 4, row,
 *             offset low, offset high));  class = argmax_c [ log2 W_c - log2(-log2 v_c) ], ties to the lowest c
 *   level 2:  u_j = uniform(word j % 4 of counter (j / 4, row, offset low, offset high));
 *             token = argmax over the class's j of [ y_j - log2(-log2 u_j) ], ties to the lowest j
 *   Element j is drawn with probability softmax(logits / temperature)_j; only the winning class needs its
 *   elements' uniforms, which is why the call runs at the speed of ppo_logprob_entropy.
 * Use a new `offset` for every call that must be independent of the previous ones with the same seed.
 *   logits [rows, V] dtype, row pitch row_stride >= V elements
 *   tokens_out [rows] i32; logprob, entropy, lse nullable [rows] f32 (as in ppo_logprob_entropy)
 *   workspace  nullable (status word: PPO_DEV_BAD_ROW when a row has a NaN, a +inf or no finite logit;
 *              that row gets token -1 and NaN outputs)
 * The kernel evaluates the rule in fp32 with hardware exp2/log2 approximations: where two candidates'
 * scores differ by less than ~1e-5 it may pick the other one than an exact evaluation would.
 */
int ppo_sample_logprob_entropy(const void *logits, int dtype, int64_t rows, int64_t V, int64_t row_stride,
                               float temperature, uint64_t seed, uint64_t offset, int32_t *tokens_out,
                               float *logprob, float *entropy, float *lse, void *workspace, void *stream);

/*
 * Chain rule from token log-probs back to the logits (the backward half of ppo_logprob_entropy;
 * used by losses that are functions of sequence log-probs, such as the DPO loss below):
 *   dlogits[r, j] = dlogprob[r] * (1[j == tokens[r]] - softmax(logits[r, :] / temperature)[j]) / temperature
 * for rows with mask[r] != 0; rows with mask 0 are zero-filled and their logits are never read.
 *   logits   [rows, V] dtype, contiguous (row pitch V);  dlogits [rows, V] same dtype, != logits
 *   tokens   [rows] i32;  mask [rows] u8;  dlogprob [rows] f32 (upstream gradient)
 *   new_logprob, entropy  nullable [rows] f32 outputs: the row's log-prob / entropy, recomputed on the way
 *   workspace  required, >= ppo_workspace_bytes(rows, 1, V), 256-byte aligned
 * One read of the real rows and one write of all rows (same kernels as ppo_loss_fwd_bwd).  A token id
 * outside [0, V) makes its row NaN and sets PPO_DEV_BAD_TOKEN.
 */
int ppo_logprob_bwd(const void *logits, int dtype, int64_t rows, int64_t V, const int32_t *tokens,
                    const uint8_t *mask, const float *dlogprob, float temperature, void *dlogits,
                    float *new_logprob, float *entropy, void *workspace, void *stream);

/*
 * Reward-model loss (section "Preliminaries", step 2): mean over the P pairs of
 * -log sigma(r_chosen - r_rejected) = log(1 + e^(r_rejected - r_chosen)).
 *   reward_chosen, reward_rejected  [P] f32
 *   out4  [4] f32: loss, accuracy (share of pairs with r_chosen > r_rejected), mean r_chosen, mean r_rejected
 *   dreward_chosen, dreward_rejected  nullable [P] f32: gradient of the mean loss
 * One block, fp64 sums in a fixed order.  No workspace.
 */
int ppo_pairwise_loss(const float *reward_chosen, const float *reward_rejected, int64_t P, float *out4,
                      float *dreward_chosen, float *dreward_rejected, void *stream);

/*
 * DPO loss (section "Preliminaries", "RL-free approaches") from token log-probs of the chosen and
 * the rejected completion under the policy and under the frozen SFT reference:
 *   reward = beta * (sum_t mask * logprob - sum_t mask * ref_logprob)       (the implicit reward)
 *   loss   = mean over pairs of -log sigma(reward_chosen - reward_rejected)
 *   logprob_*, ref_logprob_*  [P, T] f32;  mask_*  [P, T] u8 (1 on response tokens)
 *   out4  [4] f32: loss, accuracy of the implicit rewards, mean reward_chosen, mean reward_rejected
 *   reward_chosen, reward_rejected  nullable [P] f32
 *   dlogprob_chosen, dlogprob_rejected  nullable [P, T] f32: gradient of the mean loss w.r.t. the
 *       policy's token log-probs (0 outside the mask); feed them to ppo_logprob_bwd
 * beta: Table "DPO hyperparameters" (0.05).  One block, one warp per pair, fp64 sums in a fixed order.
 */
int ppo_dpo_loss(const float *logprob_chosen, const float *logprob_rejected, const float *ref_logprob_chosen,
                 const float *ref_logprob_rejected, const uint8_t *mask_chosen, const uint8_t *mask_rejected,
                 int64_t P, int32_t T, float beta, float *out4, float *reward_chosen, float *reward_rejected,
                 float *dlogprob_chosen, float *dlogprob_rejected, void *stream);

/*
 * Allocation-free variant of ppo_loss_from_logprob (an addition of this library; the paper has no
 * counterpart).  It is meant for callers that cannot obtain device memory at the point of the call:
 * code running under a framework whose allocator must not be re-entered, inside a region where
 * cudaMalloc is forbidden or would synchronise the device, or in a process whose memory budget
 * has been handed out in full.  Its scratch (what the other entry point takes as `workspace`) is
 * a fixed array built into the library: 256 + 36 * PPO_STATIC_MAX_TOKENS bytes (about 1.2 MB) of
 * device memory on every GPU that loads the library, held until the process exits.
 *   - Same arguments, results and error codes as ppo_loss_from_logprob, minus `workspace`;
 *     B*T > PPO_STATIC_MAX_TOKENS returns PPO_ERR_UNSUPPORTED before anything is launched.
 *   - Neither this call nor anything it uses calls cudaMalloc, cudaFree or an allocating library
 *     routine.  The first call on each device looks up the array's device address (with that
 *     device current); make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the last call's contents; each call rewrites what
 *     it reads and clears the status word itself.  Two calls that overlap on the same GPU (different
 *     streams, or different host threads) race on it: serialise them.
 *   - There is no status word to read back; an all-zero mask shows as losses[PPO_LOSS_N] == 0.
 */
#define PPO_STATIC_MAX_TOKENS 32768
int ppo_loss_from_logprob_static(const float *new_logprob, const float *entropy, int32_t B, int32_t T,
                                 const uint8_t *mask, const float *old_logprob, const float *advantages,
                                 const float *values_new, const float *values_old, const float *returns,
                                 const ppo_params *p /* host */, float *losses, float *dlogprob,
                                 float *dvalues, void *stream);

/*
 * Step 7 (fused LM head): logits[r, :] = H[r, :] . W are formed tile by tile on the tensor
 * cores (bf16 inputs, fp32 accumulation in tensor memory) and consumed by step 1's reduction
 * in the epilogue; they are never written to memory.
 *   H [M,K] bf16 row-major;  W [K,V] bf16 row-major;  tokens [M];  mask nullable [M]
 *   logprob [M] f32;  entropy, lse nullable [M] f32
 * Rows with mask 0 output 0 and are taken out of the multiplication: the rows with mask 1 are packed
 * into the workspace first (their number is found on the device) and only those are multiplied;
 * the results are those of the call without a mask on these rows, bit for bit.
 * Requirements: K % 64 == 0, V % 8 == 0, H and W 16-byte aligned; otherwise
 * PPO_ERR_UNSUPPORTED.  workspace required (ppo_lmhead_workspace_bytes: per-row partial results,
 * the row order and room for the packed copy of H, M*K*2 bytes).
 */
int ppo_lmhead_logprob_entropy(const void *H, const void *W, int64_t M, int64_t K, int64_t V,
                               const int32_t *tokens, const uint8_t *mask, float temperature,
                               float *logprob, float *entropy, float *lse, void *workspace,
                               void *stream);

/*
 * Backward of the fused LM head (the step after ppo_loss_from_logprob when the logits were never
 * materialised): with z = H W / temperature and the gradient g = dlogprob on each token's log-prob,
 *   dlogits = g * (onehot(token) - softmax(z)) / temperature   [M, V]
 *   dH = dlogits W^T  [M, K],   dW = H^T dlogits  [K, V]
 * Three tensor-core passes: the logits are recomputed tile by tile and turned into dlogits in the
 * epilogue (using the log-sum-exp saved by ppo_lmhead_logprob_entropy), then two contractions.
 *   H [M,K], W [K,V]  bf16 as in ppo_lmhead_logprob_entropy;  tokens [M] i32;  mask nullable [M] u8
 *   lse [M] f32       the `lse` output of ppo_lmhead_logprob_entropy for the same H, W, temperature
 *   dlogprob [M] f32  upstream gradient (rows with mask 0 or dlogprob 0 give zero rows)
 *   dlogits [M,V] bf16  required scratch AND output: the only intermediate written to memory.
 *                       Without a mask, or with M <= 128: every row at its place.  With a mask and
 *                       M > 128 the rows with mask 0 are taken out of all three passes, and the
 *                       buffer returns the gradient rows of the rows with mask 1 PACKED at its
 *                       front, in row order (the rest of it is scratch)
 *   dH [M,K], dW [K,V]  bf16 outputs, each nullable (its pass is skipped); rows of dH with mask 0
 *                       are 0
 *   workspace  required, ppo_lmhead_workspace_bytes(M, K, V) bytes (status word, row order, packed
 *              copy of H), 256-byte aligned
 * Requirements: K % 8 == 0, V % 8 == 0, all matrices 16-byte aligned; else PPO_ERR_UNSUPPORTED /
 * PPO_ERR_ALIGN.  Token ids are assumed valid (the forward call reports bad ones).
 */
int ppo_lmhead_bwd(const void *H, const void *W, int64_t M, int64_t K, int64_t V, const int32_t *tokens,
                   const uint8_t *mask, const float *lse, const float *dlogprob, float temperature,
                   void *dlogits, void *dH, void *dW, void *workspace, void *stream);

/*
 * The whole path in one call.  ppo_step_io names every buffer of one PPO iteration over a batch of
 * B responses x T tokens; all pointers of one struct live in the same memory space.
 *   inputs   policy_logits, ref_logits [B,T,V] (dtype); loss_logits [B,T,V] or NULL (= policy_logits);
 *            responses [B,T] i32; scores [B]; values, values_new [B,T];
 *            old_logprob [B,T] or NULL (= the log-probs this call computes: first PPO epoch, ratio 1)
 *   outputs  responses_out, eos_index, seq_len, mask, scores_out (step 2); logprob, entropy,
 *            ref_logprob (step 1, as with the mask of step 2: 0 at the padding positions after a
 *            response's first EOS, whose logits are not read); kl, rewards (step 3; with params.whiten_rewards the rewards
 *            array holds the whitened rewards that GAE consumed); advantages, returns (step 4);
 *            advantages_whitened, whiten_stats[3] (step 5); losses[8], dlogits, dvalues and the
 *            nullable new_logprob, new_entropy, dlogprob (step 6); workspace (device only)
 *
 * ppo_step: `io` is a host struct of DEVICE pointers; runs steps 1 (policy and reference), 2, 3, 4,
 * 5, 6 on `stream` without synchronising; its launches overlap where their inputs allow (the loss
 * kernel starts while the token-level kernel runs, the token-level kernel while the log-prob kernel
 * drains), so no output buffer may alias an input buffer or another output buffer, and one
 * workspace serves one call at a time.  Errors are those of the individual calls.
 *
 * ppo_step_host: `host` is a host struct of HOST pointers (pinned memory makes the copies
 * asynchronous), `dev` a host struct of DEVICE pointers used as staging and output buffers.  Copies
 * every input host -> device (of the logits tensors only the rows ppo_step reads: each response's
 * positions up to its first EOS, found from host->responses; the other rows of the staging buffers
 * are left as they are), runs ppo_step on `dev`, copies back each output whose pointer in
 * `host` is not NULL, and waits for the stream.  Inputs that are NULL in `host` (loss_logits,
 * old_logprob) are treated as in ppo_step.  The copies of the reference tensor are queued on a
 * side stream of the library (one per device, created by the first call on that device and kept
 * until the process exits) that is ordered after the work already in `stream` and before the
 * kernels of this call, so that two copy queues keep the host link busy; the call is safe from
 * several host threads.
 */
typedef struct ppo_step_io {
    const void *policy_logits, *ref_logits, *loss_logits;
    const int32_t *responses;
    const float *scores, *values, *values_new, *old_logprob;
    int32_t *responses_out, *eos_index, *seq_len;
    uint8_t *mask;
    float *scores_out, *logprob, *entropy, *ref_logprob, *kl, *rewards, *advantages, *returns,
        *advantages_whitened, *whiten_stats, *losses;
    void *dlogits;
    float *dvalues, *new_logprob, *new_entropy, *dlogprob;
    void *workspace;
} ppo_step_io;

int ppo_step(const ppo_step_io *io /* host */, int dtype, int32_t B, int32_t T, int64_t V,
             const ppo_params *p /* host */, void *stream);
int ppo_step_host(const ppo_step_io *host /* host */, const ppo_step_io *dev /* host */, int dtype,
                  int32_t B, int32_t T, int64_t V, const ppo_params *p /* host */, void *stream);

/*
 * The config with the fused LM head as one call: the logits are never materialised, so the path is
 * steps 2 (EOS trick), 1 through ppo_lmhead_logprob_entropy for the policy unembedding W and for the frozen
 * SFT reference's W_ref (both with the mask of step 2: padding rows are taken out of the GEMMs), 3, 4, 5 and
 * step 6 at log-prob level (ppo_loss_from_logprob).  Same citations as the individual calls.
 *   inputs   H [B*T, K] bf16 hidden states of the response positions; W, W_ref [K, V] bf16;
 *            responses [B,T] i32; scores [B]; values, values_new [B,T];
 *            old_logprob [B,T] or NULL (= the log-probs this call computes: first PPO epoch, ratio 1)
 *   outputs  responses_out, eos_index, seq_len, mask, scores_out; logprob, entropy, lse, ref_logprob (0 at
 *            padding positions); kl, rewards; advantages, returns; advantages_whitened, whiten_stats[3];
 *            losses[8], dlogprob, dvalues; workspace (device only) of at least
 *            max(ppo_lmhead_workspace_bytes(B*T, K, V), ppo_workspace_bytes(B, T, V)) bytes
 * ppo_lmhead_step: `io` is a host struct of DEVICE pointers; everything is enqueued on `stream`, nothing
 * synchronises.  K a multiple of 64, V a multiple of 8 (PPO_ERR_UNSUPPORTED otherwise).
 * ppo_lmhead_step_host: `host` holds HOST pointers (pinned memory makes the copies asynchronous), `dev` the
 * device staging and output buffers.  Copies the inputs host -> device (of H only the rows the GEMMs read:
 * each response's positions up to its first EOS, found from host->responses), runs ppo_lmhead_step on `dev`,
 * copies back each output whose pointer in `host` is not NULL and waits for the stream.
 */
typedef struct ppo_lmhead_step_io {
    const void *H, *W, *W_ref;
    const int32_t *responses;
    const float *scores, *values, *values_new, *old_logprob;
    int32_t *responses_out, *eos_index, *seq_len;
    uint8_t *mask;
    float *scores_out, *logprob, *entropy, *lse, *ref_logprob, *kl, *rewards, *advantages, *returns,
        *advantages_whitened, *whiten_stats, *losses, *dlogprob, *dvalues;
    void *workspace;
} ppo_lmhead_step_io;

int ppo_lmhead_step(const ppo_lmhead_step_io *io /* host */, int32_t B, int32_t T, int64_t K, int64_t V,
                    const ppo_params *p /* host */, void *stream);
int ppo_lmhead_step_host(const ppo_lmhead_step_io *host /* host */, const ppo_lmhead_step_io *dev /* host */,
                         int32_t B, int32_t T, int64_t K, int64_t V, const ppo_params *p /* host */, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PPO_B200_H */
