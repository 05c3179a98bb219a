// Preference losses on sequence log-probabilities (section "Preliminaries" of the paper): the reward
// model's pairwise logistic loss, and the DPO loss with its implicit rewards. Both are tiny,
// latency-bound reductions over the pairs of a batch (fp64 sums in a fixed order); the heavy part of a
// DPO step - token log-probs from the logits, and the gradient back to the logits - is done by
// ppo_logprob_entropy and ppo_logprob_bwd.
#include "ppo_common.cuh"

namespace ppo {

constexpr int kPrefThreads = 1024;

// -log sigma(d) = log(1 + e^(-d)) and sigma(-d) = 1 / (1 + e^d), without overflow for large |d|
__device__ __forceinline__ void logistic_terms(double d, double &loss, double &sig_neg)
{
    const double e = exp(-fabs(d));            // in (0, 1]
    loss = log1p(e) + (d < 0.0 ? -d : 0.0);
    sig_neg = d >= 0.0 ? e / (1.0 + e) : 1.0 / (1.0 + e);
}

// One block. Thread t owns pairs t, t + 1024, ...: loss, accuracy and mean rewards are block sums of
// the per-thread fp64 partial sums; the gradient of the MEAN loss is written per pair.
__global__ void __launch_bounds__(kPrefThreads)
pairwise_loss_kernel(const float *__restrict__ r_c, const float *__restrict__ r_r, int64_t P,
                     float *__restrict__ out4, float *__restrict__ dr_c, float *__restrict__ dr_r)
{
    __shared__ double red[32];
    double s_loss = 0.0, s_acc = 0.0, s_c = 0.0, s_r = 0.0;
    const double inv_p = 1.0 / (double)P;
    for (int64_t i = threadIdx.x; i < P; i += kPrefThreads) {
        const double c = (double)r_c[i], r = (double)r_r[i];
        double loss, sn;
        logistic_terms(c - r, loss, sn);
        s_loss += loss;
        s_acc += c > r ? 1.0 : 0.0;
        s_c += c;
        s_r += r;
        if (dr_c) dr_c[i] = (float)(-sn * inv_p);
        if (dr_r) dr_r[i] = (float)(sn * inv_p);
    }
    s_loss = block_sum<kPrefThreads>(s_loss, red);
    s_acc = block_sum<kPrefThreads>(s_acc, red);
    s_c = block_sum<kPrefThreads>(s_c, red);
    s_r = block_sum<kPrefThreads>(s_r, red);
    if (threadIdx.x == 0) {
        out4[0] = (float)(s_loss * inv_p);
        out4[1] = (float)(s_acc * inv_p);
        out4[2] = (float)(s_c * inv_p);
        out4[3] = (float)(s_r * inv_p);
    }
}

// sum over the response tokens of one sequence by one warp (lane-strided, then a butterfly: fixed order)
__device__ __forceinline__ double masked_sum(const float *__restrict__ x, const uint8_t *__restrict__ m, int T, int lane)
{
    double s = 0.0;
    for (int t = lane; t < T; t += 32)
        if (m[t]) s += (double)x[t];
    return warp_sum(s);
}

// One block. Four warps share a pair (one masked sequence sum each: policy / reference x chosen / rejected), so
// eight pairs are in flight per round; then each of the four computes the pair's terms from the four sums and two
// of them write the per-token gradient of the MEAN loss w.r.t. the policy's token log-probs (chosen, rejected).
__global__ void __launch_bounds__(kPrefThreads)
dpo_loss_kernel(const float *__restrict__ lp_c, const float *__restrict__ lp_r, const float *__restrict__ ref_c,
                const float *__restrict__ ref_r, const uint8_t *__restrict__ mask_c,
                const uint8_t *__restrict__ mask_r, int64_t P, int T, double beta, float *__restrict__ out4,
                float *__restrict__ reward_c, float *__restrict__ reward_r, float *__restrict__ dlp_c,
                float *__restrict__ dlp_r)
{
    __shared__ double red[32];
    __shared__ double sums[kPrefThreads / 128][4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int slot = warp >> 2, part = warp & 3;
    const double inv_p = 1.0 / (double)P;
    double s_loss = 0.0, s_acc = 0.0, s_c = 0.0, s_r = 0.0;   // partial sums, carried by the `part == 0` warps
    for (int64_t i0 = 0; i0 < P; i0 += kPrefThreads / 128) {
        const int64_t i = i0 + slot;
        const int64_t o = i * T;
        if (i < P) {
            const float *x = part == 0 ? lp_c : (part == 1 ? ref_c : (part == 2 ? lp_r : ref_r));
            const uint8_t *m = part < 2 ? mask_c : mask_r;
            const double v = masked_sum(x + o, m + o, T, lane);
            if (lane == 0) sums[slot][part] = v;
        }
        __syncthreads();
        if (i < P) {
            const double rc = beta * (sums[slot][0] - sums[slot][1]);
            const double rr = beta * (sums[slot][2] - sums[slot][3]);
            double loss, sn;
            logistic_terms(rc - rr, loss, sn);
            if (part == 0) {
                s_loss += loss;
                s_acc += rc > rr ? 1.0 : 0.0;
                s_c += rc;
                s_r += rr;
                if (lane == 0) {
                    if (reward_c) reward_c[i] = (float)rc;
                    if (reward_r) reward_r[i] = (float)rr;
                }
                if (dlp_c) {
                    const float gc = (float)(-beta * sn * inv_p);
                    for (int t = lane; t < T; t += 32) dlp_c[o + t] = mask_c[o + t] ? gc : 0.f;
                }
            } else if (part == 2 && dlp_r) {
                const float gr = (float)(beta * sn * inv_p);
                for (int t = lane; t < T; t += 32) dlp_r[o + t] = mask_r[o + t] ? gr : 0.f;
            }
        }
        __syncthreads();   // sums[] is rewritten in the next round
    }
    // one lane of every `part == 0` warp carries that warp's sums into the block sums
    const double keep = (lane == 0 && part == 0) ? 1.0 : 0.0;
    s_loss = block_sum<kPrefThreads>(s_loss * keep, red);
    s_acc = block_sum<kPrefThreads>(s_acc * keep, red);
    s_c = block_sum<kPrefThreads>(s_c * keep, red);
    s_r = block_sum<kPrefThreads>(s_r * keep, red);
    if (threadIdx.x == 0) {
        out4[0] = (float)(s_loss * inv_p);
        out4[1] = (float)(s_acc * inv_p);
        out4[2] = (float)(s_c * inv_p);
        out4[3] = (float)(s_r * inv_p);
    }
}

}   // namespace ppo

using namespace ppo;

extern "C" int ppo_pairwise_loss(const float *reward_chosen, const float *reward_rejected, int64_t P, float *out4,
                                 float *dreward_chosen, float *dreward_rejected, void *stream)
{
    if (P <= 0 || P >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    if (!reward_chosen || !reward_rejected || !out4) return PPO_ERR_NULL;
    pairwise_loss_kernel<<<1, kPrefThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        reward_chosen, reward_rejected, P, out4, dreward_chosen, dreward_rejected);
    return launch_status();
}

extern "C" int ppo_dpo_loss(const float *logprob_chosen, const float *logprob_rejected, const float *ref_logprob_chosen,
                            const float *ref_logprob_rejected, const uint8_t *mask_chosen,
                            const uint8_t *mask_rejected, int64_t P, int32_t T, float beta, float *out4,
                            float *reward_chosen, float *reward_rejected, float *dlogprob_chosen,
                            float *dlogprob_rejected, void *stream)
{
    if (P <= 0 || T <= 0 || P * (int64_t)T >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    if (!logprob_chosen || !logprob_rejected || !ref_logprob_chosen || !ref_logprob_rejected || !mask_chosen ||
        !mask_rejected || !out4)
        return PPO_ERR_NULL;
    if (!finite_f(beta)) return PPO_ERR_PARAM;
    dpo_loss_kernel<<<1, kPrefThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        logprob_chosen, logprob_rejected, ref_logprob_chosen, ref_logprob_rejected, mask_chosen, mask_rejected, P, T,
        (double)beta, out4, reward_chosen, reward_rejected, dlogprob_chosen, dlogprob_rejected);
    return launch_status();
}
