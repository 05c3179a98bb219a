/*
 * ppo_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the per-token PPO-for-RLHF path of arXiv 2403.17031
 * ("The N+ Implementation Details of RLHF with PPO").  It exists so the CUDA library can be
 * checked against something written independently of it: it shares no code, header, table
 * or helper with the CUDA sources, and nothing in the product may call it.  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg load it.
 *
 * Every function is the textbook definition written out: three explicit passes per softmax
 * row (max, sum, entropy), a sequential reverse loop for GAE, two-pass mean/variance.  The
 * only parallelism is an OpenMP "for" over independent rows.  Stored inputs (fp32 or bf16
 * bit patterns) are widened exactly to double before any arithmetic.
 *
 * Where the paper states hyper-parameters but prints no formula (log-softmax gather,
 * entropy, the k1 KL estimator, GAE, the clipped losses) the standard definitions are used;
 * each function names the passage it follows and the reading taken.
 *
 * Pins (all in tests/, none of them calls the CUDA path): uniform rows, the one-hot closed
 * form, shift invariance, brute force on tiny V, float64 library log-softmax at tau = 1,
 * hand-enumerated EOS rows, GAE closed forms (lambda = gamma = 1; lambda = 0; O(T^2) sum;
 * a hand case), the paper's whiten() listing evaluated with a CPU array library, ratio = 1
 * and v = v_old special cases, and central finite differences of the oracle's own loss.
 * The fused LM-head function is pinned by a library float64 matmul followed by a library
 * log-softmax.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* conventions the paper does not print; named so that another reading is a one-line change */
#define VALUE_LOSS_FACTOR 0.5   /* vf_loss = VALUE_LOSS_FACTOR * masked_mean(max(...)) */

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* One softmax row: z_j = x_j / tau, lse = log sum_j exp(z_j), H = -sum_j p_j log p_j.
 * Three passes, exactly as the definition reads. Entries equal to -inf carry probability 0
 * and add nothing to H. */
static void softmax_row_stats(const void *logits, int dtype, int64_t off, int64_t V, double tau,
                              double *lse_out, double *H_out)
{
    double M = -INFINITY;
    for (int64_t j = 0; j < V; ++j) {
        double z = widen(logits, dtype, off + j) / tau;
        if (z > M) M = z;
    }
    double S = 0.0;
    for (int64_t j = 0; j < V; ++j) {
        double z = widen(logits, dtype, off + j) / tau;
        S += exp(z - M);
    }
    double lse = M + log(S);
    double H = 0.0;
    for (int64_t j = 0; j < V; ++j) {
        double z = widen(logits, dtype, off + j) / tau;
        if (z == -INFINITY) continue;
        double logp = z - lse;
        H -= exp(logp) * logp;
    }
    *lse_out = lse;
    *H_out = H;
}

/*
 * Step 1 -- log-probability of the sampled token and entropy of the temperature-scaled
 * distribution, for each row of [rows, V] logits.  The paper fixes only the temperature
 * (Table "PPO hyperparameters": sampling temperature 0.7) and that policy and SFT reference
 * are scored the same way (Eq. "RL": KL between pi_theta and pi_SFT; section "Disable dropout":
 * ratios are 1 in the first epoch, so rollout and training log-probs use one scaling).
 * Reading: z = logits / tau for both models; rows with mask 0 output 0; a token id outside
 * [0, V) yields NaN for that row.
 */
int oracle_logprob_entropy(const void *logits, int dtype, int64_t rows, int64_t V, int64_t row_stride,
                           const int32_t *tokens, const uint8_t *mask, double temperature,
                           double *logprob, double *entropy, double *lse)
{
    if (!logits || !tokens || !logprob || rows < 0 || V <= 0 || !(temperature > 0.0)) return -1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
        double lp = 0.0, H = 0.0, L = 0.0;
        if (!mask || mask[r]) {
            int64_t tok = tokens[r];
            if (tok < 0 || tok >= V) {
                lp = H = L = NAN;
            } else {
                softmax_row_stats(logits, dtype, r * row_stride, V, temperature, &L, &H);
                lp = widen(logits, dtype, r * row_stride + tok) / temperature - L;
            }
        }
        logprob[r] = lp;
        if (entropy) entropy[r] = H;
        if (lse) lse[r] = L;
    }
    return 0;
}

/*
 * Step 2 -- the "EOS trick" (section "PPO Training -> EOS trick"): a fixed number of tokens is
 * sampled; the response is cut at its first EOS and everything after it becomes [PAD]; a
 * response with no EOS has its reward-model score replaced by a constant (-1).  EOS and [PAD]
 * are distinct ids (section "Dataset -> ... do not use EOS synonymously as [PAD]").
 * Reading: the EOS token itself stays a real token (the reward is read on it, section "RM
 * Training -> Extract reward from the EOS token"); seq_len = eos_index + 1, or T with no EOS.
 */
int oracle_truncate_and_score(const int32_t *responses, int32_t B, int32_t T, int32_t eos_id,
                              int32_t pad_id, const double *scores, double no_eos_score,
                              int32_t *responses_out, int32_t *eos_index, int32_t *seq_len,
                              uint8_t *mask, double *scores_out)
{
    if (!responses || B < 0 || T <= 0 || eos_id == pad_id) return -1;
    for (int32_t b = 0; b < B; ++b) {
        int32_t e = -1;
        for (int32_t t = 0; t < T; ++t) {
            if (responses[(int64_t)b * T + t] == eos_id) { e = t; break; }
        }
        int32_t L = (e >= 0) ? e + 1 : T;
        for (int32_t t = 0; t < T; ++t) {
            int64_t i = (int64_t)b * T + t;
            if (responses_out) responses_out[i] = (t < L) ? responses[i] : pad_id;
            if (mask) mask[i] = (uint8_t)(t < L);
        }
        if (eos_index) eos_index[b] = e;
        if (seq_len) seq_len[b] = L;
        if (scores_out && scores) scores_out[b] = (e >= 0) ? scores[b] : no_eos_score;
    }
    return 0;
}

/*
 * Step 3 -- per-token reward (Eq. "RL": R = r_phi - beta * KL[pi_theta || pi_SFT]; figure
 * "reward vs value": every entry of the reward vector is a per-token KL penalty and the
 * reward-model score sits on the EOS token).  Reading: the per-token KL estimate is the
 * log-ratio at the sampled token (k1); the score is added on the last real token.
 */
int oracle_kl_rewards(const double *logprob, const double *ref_logprob, const uint8_t *mask,
                      const int32_t *seq_len, const double *scores, int32_t B, int32_t T,
                      double kl_coef, double *kl, double *rewards)
{
    if (!logprob || !ref_logprob || !mask || !seq_len || !scores || B < 0 || T <= 0) return -1;
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t t = 0; t < T; ++t) {
            int64_t i = (int64_t)b * T + t;
            double k = mask[i] ? (logprob[i] - ref_logprob[i]) : 0.0;
            if (kl) kl[i] = k;
            if (rewards) rewards[i] = mask[i] ? -kl_coef * k : 0.0;
        }
        int32_t L = seq_len[b];
        if (rewards && L >= 1 && L <= T) rewards[(int64_t)b * T + (L - 1)] += scores[b];
    }
    return 0;
}

/*
 * Step 4 -- generalised advantage estimation with the table's gamma and lambda.  The paper
 * prints no recurrence; it says the value function predicts the end-of-episode return at each
 * token (section "Value model initializes from the reward model"), so the episode ends after
 * the last real token and nothing is bootstrapped beyond it.
 *   delta_t = r_t + gamma * V_{t+1} - V_t,   A_t = delta_t + gamma * lambda * A_{t+1},
 *   return_t = A_t + V_t,   with V_{L} = A_{L} = 0 and zeros written for t >= L.
 */
int oracle_gae(const double *rewards, const double *values, const int32_t *seq_len, int32_t B,
               int32_t T, double gamma, double lam, double *advantages, double *returns)
{
    if (!rewards || !values || !seq_len || !advantages || !returns || B < 0 || T <= 0) return -1;
    for (int32_t b = 0; b < B; ++b) {
        int32_t L = seq_len[b];
        if (L < 0) L = 0;
        if (L > T) L = T;
        for (int32_t t = L; t < T; ++t) {
            advantages[(int64_t)b * T + t] = 0.0;
            returns[(int64_t)b * T + t] = 0.0;
        }
        double A_next = 0.0;
        for (int32_t t = L - 1; t >= 0; --t) {
            int64_t i = (int64_t)b * T + t;
            double V_next = (t + 1 < L) ? values[i + 1] : 0.0;
            double delta = rewards[i] + gamma * V_next - values[i];
            double A = delta + gamma * lam * A_next;
            advantages[i] = A;
            returns[i] = A + values[i];
            A_next = A;
        }
    }
    return 0;
}

/*
 * Step 5 -- the paper's whiten() (section "Reward whitening" listing; used on advantages in
 * section "Advantage whitening") restricted to the entries with mask 1: biased variance,
 * division by sqrt(var + eps) with eps = 1e-8; shift_mean != 0 leaves the result centred at
 * zero, shift_mean == 0 adds the mean back.  Entries with mask 0 are written as 0.
 * stats3 = {mean, variance, count}.  A null mask means every entry counts.
 */
int oracle_whiten(const double *x, const uint8_t *mask, int64_t n_elems, int shift_mean, double eps,
                  double *out, double *stats3)
{
    if (!x || !out || n_elems < 0) return -1;
    double n = 0.0, sum = 0.0;
    for (int64_t i = 0; i < n_elems; ++i)
        if (!mask || mask[i]) { n += 1.0; sum += x[i]; }
    double mean = (n > 0.0) ? sum / n : 0.0;
    double ss = 0.0;
    for (int64_t i = 0; i < n_elems; ++i)
        if (!mask || mask[i]) { double d = x[i] - mean; ss += d * d; }
    double var = (n > 0.0) ? ss / n : 0.0;
    double inv = 1.0 / sqrt(var + eps);
    for (int64_t i = 0; i < n_elems; ++i) {
        if (!mask || mask[i]) {
            double y = (x[i] - mean) * inv;
            if (!shift_mean) y += mean;
            out[i] = y;
        } else {
            out[i] = 0.0;
        }
    }
    if (stats3) { stats3[0] = mean; stats3[1] = var; stats3[2] = n; }
    return 0;
}

/*
 * Step 6 -- clipped PPO policy loss and clipped value loss (Table "PPO hyperparameters":
 * epsilon = 0.2, epsilon-hat = 0.2, c1 = 0.1, value-loss clipping on, one minibatch), with
 * their analytic gradients.  The paper prints the hyper-parameters only; the formulas are
 * the standard ones:
 *   rho = exp(lp_new - lp_old)
 *   pg  = max(-A*rho, -A*clip(rho, 1-eps, 1+eps))
 *   vc  = clip(v, v_old - epsv, v_old + epsv);  vf = max((v-ret)^2, (vc-ret)^2)
 *   pg_loss = sum(m*pg)/n; vf_loss = VALUE_LOSS_FACTOR*sum(m*vf)/n; loss = pg_loss + c1*vf_loss
 * Readings: masked mean over the n real tokens; entropy is a statistic only (the table has no
 * entropy coefficient); a clipped branch that is strictly larger stops the gradient.
 *   d loss / d lp_new = (m/n) * (-A*rho)           when the unclipped branch is the max
 *   d loss / d logit_j = dlp * (1[j = tok] - p_j) / tau
 *   d loss / d v = c1 * 2*VALUE_LOSS_FACTOR * (m/n) * (v - ret)   when (v-ret)^2 >= (vc-ret)^2
 *
 * losses[8] = {pg_loss, vf_loss, loss, approx_kl = 0.5*mean((lp_new-lp_old)^2), pg_clipfrac,
 *              vf_clipfrac, mean entropy, n}.
 * dlogits (nullable): if sel_rows is null it is [rows, V]; otherwise [n_sel, V] holding the
 * rows listed in sel_rows.  dlogprob (nullable) receives d loss / d lp_new per token.
 */
int oracle_loss_fwd_bwd(const void *logits, int dtype, int32_t B, int32_t T, int64_t V,
                        const int32_t *tokens, const uint8_t *mask, const double *old_logprob,
                        const double *advantages, const double *values_new, const double *values_old,
                        const double *returns, double temperature, double cliprange,
                        double cliprange_value, double vf_coef, double *losses, double *dlogits,
                        const int64_t *sel_rows, int64_t n_sel, double *dvalues, double *new_logprob,
                        double *entropy, double *dlogprob)
{
    if (!logits || !tokens || !mask || !old_logprob || !advantages || !values_new || !values_old ||
        !returns || !losses || B <= 0 || T <= 0 || V <= 0 || !(temperature > 0.0))
        return -1;
    const int64_t rows = (int64_t)B * T;
    double n = 0.0;
    for (int64_t r = 0; r < rows; ++r) n += mask[r] ? 1.0 : 0.0;
    double pg_sum = 0, vf_sum = 0, kl_sum = 0, pgc = 0, vfc = 0, ent_sum = 0;
    const int64_t n_out = (dlogits && sel_rows) ? n_sel : (dlogits ? rows : 0);

    /* per-token quantities first (sequential accumulation, fixed order) */
    for (int64_t r = 0; r < rows; ++r) {
        if (dvalues) dvalues[r] = 0.0;
        if (new_logprob) new_logprob[r] = 0.0;
        if (entropy) entropy[r] = 0.0;
        if (dlogprob) dlogprob[r] = 0.0;
    }
    /* softmax statistics of each real row (the expensive part; rows are independent) */
    /* storage for per-row results only: no blocking, no fusion */
    double *lse_buf = (double *)malloc(sizeof(double) * (size_t)rows);
    double *ent_buf = (double *)malloc(sizeof(double) * (size_t)rows);
    if (!lse_buf || !ent_buf) { free(lse_buf); free(ent_buf); return -2; }
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
        lse_buf[r] = 0.0;
        ent_buf[r] = 0.0;
        if (mask[r] && tokens[r] >= 0 && tokens[r] < V)
            softmax_row_stats(logits, dtype, r * V, V, temperature, &lse_buf[r], &ent_buf[r]);
    }
    for (int64_t r = 0; r < rows; ++r) {
        if (!mask[r]) continue;
        int64_t tok = tokens[r];
        double lp_new = (tok >= 0 && tok < V) ? widen(logits, dtype, r * V + tok) / temperature - lse_buf[r]
                                              : NAN;
        double A = advantages[r];
        double logratio = lp_new - old_logprob[r];
        double rho = exp(logratio);
        double rho_c = rho < 1.0 - cliprange ? 1.0 - cliprange : (rho > 1.0 + cliprange ? 1.0 + cliprange : rho);
        double l1 = -A * rho, l2 = -A * rho_c;
        double pg = l1 > l2 ? l1 : l2;
        double v = values_new[r], vo = values_old[r], ret = returns[r];
        double lo = vo - cliprange_value, hi = vo + cliprange_value;
        double vc = v < lo ? lo : (v > hi ? hi : v);
        double e1 = (v - ret) * (v - ret), e2 = (vc - ret) * (vc - ret);
        double vf = e1 > e2 ? e1 : e2;
        pg_sum += pg;
        vf_sum += vf;
        kl_sum += 0.5 * logratio * logratio;
        pgc += (l2 > l1) ? 1.0 : 0.0;
        vfc += (e2 > e1) ? 1.0 : 0.0;
        ent_sum += ent_buf[r];
        double glp = (l2 > l1) ? 0.0 : (-A * rho) / n;
        if (dlogprob) dlogprob[r] = glp;
        if (dvalues) dvalues[r] = (e2 > e1) ? 0.0 : vf_coef * 2.0 * VALUE_LOSS_FACTOR * (v - ret) / n;
        if (new_logprob) new_logprob[r] = lp_new;
        if (entropy) entropy[r] = ent_buf[r];
    }
    losses[0] = n > 0 ? pg_sum / n : 0.0;
    losses[1] = n > 0 ? VALUE_LOSS_FACTOR * vf_sum / n : 0.0;
    losses[2] = losses[0] + vf_coef * losses[1];
    losses[3] = n > 0 ? kl_sum / n : 0.0;
    losses[4] = n > 0 ? pgc / n : 0.0;
    losses[5] = n > 0 ? vfc / n : 0.0;
    losses[6] = n > 0 ? ent_sum / n : 0.0;
    losses[7] = n;

    /* gradient with respect to the logits, row by row */
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t k = 0; k < n_out; ++k) {
        int64_t r = sel_rows ? sel_rows[k] : k;
        double *g = dlogits + k * V;
        if (r < 0 || r >= rows || !mask[r]) {
            for (int64_t j = 0; j < V; ++j) g[j] = 0.0;
            continue;
        }
        int64_t tok = tokens[r];
        double lp_new = widen(logits, dtype, r * V + tok) / temperature - lse_buf[r];
        double A = advantages[r];
        double rho = exp(lp_new - old_logprob[r]);
        double rho_c = rho < 1.0 - cliprange ? 1.0 - cliprange : (rho > 1.0 + cliprange ? 1.0 + cliprange : rho);
        double l1 = -A * rho, l2 = -A * rho_c;
        double glp = (l2 > l1) ? 0.0 : (-A * rho) / n;
        for (int64_t j = 0; j < V; ++j) {
            double z = widen(logits, dtype, r * V + j) / temperature;
            double p = exp(z - lse_buf[r]);
            g[j] = glp * ((j == tok ? 1.0 : 0.0) - p) / temperature;
        }
    }
    free(lse_buf);
    free(ent_buf);
    return 0;
}

/*
 * Config "fused LM head": logits row r = H[r, :] . W  (H [M,K], W [K,V], both stored bf16),
 * followed by step 1 on that row.  The logits are formed in fp64 one row at a time for the
 * rows listed in sel_rows (null = all rows); outputs are indexed by position in that list.
 */
int oracle_lmhead_logprob_entropy(const uint16_t *H, const uint16_t *W, int64_t M, int64_t K, int64_t V,
                                  const int32_t *tokens, const int64_t *sel_rows, int64_t n_sel,
                                  double temperature, double *logprob, double *entropy, double *lse)
{
    if (!H || !W || !tokens || !logprob || M <= 0 || K <= 0 || V <= 0 || !(temperature > 0.0)) return -1;
    const int64_t n_out = sel_rows ? n_sel : M;
    int err = 0;
#pragma omp parallel
    {
        double *row = (double *)malloc(sizeof(double) * (size_t)V);
        if (!row) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t k = 0; k < n_out; ++k) {
            if (!row) continue;
            int64_t r = sel_rows ? sel_rows[k] : k;
            for (int64_t j = 0; j < V; ++j) row[j] = 0.0;
            for (int64_t i = 0; i < K; ++i) {
                double h = widen(H, ORACLE_BF16, r * K + i);
                for (int64_t j = 0; j < V; ++j) row[j] += h * widen(W, ORACLE_BF16, i * V + j);
            }
            /* step 1 on the fp64 row (same three passes) */
            double Mx = -INFINITY;
            for (int64_t j = 0; j < V; ++j) { double z = row[j] / temperature; if (z > Mx) Mx = z; }
            double S = 0.0;
            for (int64_t j = 0; j < V; ++j) S += exp(row[j] / temperature - Mx);
            double L = Mx + log(S);
            double Hh = 0.0;
            for (int64_t j = 0; j < V; ++j) { double lp = row[j] / temperature - L; Hh -= exp(lp) * lp; }
            int64_t tok = tokens[r];
            logprob[k] = (tok >= 0 && tok < V) ? row[tok] / temperature - L : NAN;
            if (entropy) entropy[k] = Hh;
            if (lse) lse[k] = L;
        }
        free(row);
    }
    return err ? -2 : 0;
}
