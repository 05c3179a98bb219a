// The three statistics the paper plots for a PPO run (figure of PPO learning curves): mean RLHF reward R of Eq. "RL",
// mean over the responses of the summed per-token KL terms, mean reward-model score. [B,T]-sized work: one block, warp
// per response, fp64 sums in a fixed order (the result does not depend on scheduling).
#include "ppo_common.cuh"

using namespace ppo;

namespace {

constexpr int kCurveThreads = 1024;

__global__ void __launch_bounds__(kCurveThreads)
curves_kernel(const float *__restrict__ kl, const uint8_t *__restrict__ mask, const float *__restrict__ scores, int B,
              int T, double kl_coef, float *__restrict__ out3)
{
    __shared__ double part[3][kCurveThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double sum_R = 0.0, sum_kl = 0.0, sum_score = 0.0;       // meaningful in lane 0: this warp's responses, in order
    for (int b = warp; b < B; b += kCurveThreads / 32) {
        const float *row = kl + (int64_t)b * T;
        const uint8_t *m = mask ? mask + (int64_t)b * T : nullptr;
        double s = 0.0;
        for (int t = lane; t < T; t += 32)
            if (!m || m[t]) s += (double)row[t];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const double r = (double)scores[b];
        sum_kl += s;
        sum_score += r;
        sum_R += r - kl_coef * s;
    }
    if (lane == 0) {
        part[0][warp] = sum_R;
        part[1][warp] = sum_kl;
        part[2][warp] = sum_score;
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        double a = 0.0;
        for (int w = 0; w < kCurveThreads / 32; ++w) a += part[threadIdx.x][w];
        out3[threadIdx.x] = (float)(a / (double)B);
    }
}

}   // namespace

extern "C" int ppo_rollout_curves(const float *kl, const uint8_t *mask, const float *scores, int32_t B, int32_t T,
                                  float kl_coef, float *out3, void *stream)
{
    if (B <= 0 || T <= 0) return PPO_ERR_SHAPE;
    if (!finite_f(kl_coef)) return PPO_ERR_PARAM;
    if (!kl || !scores || !out3) return PPO_ERR_NULL;
    curves_kernel<<<1, kCurveThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(kl, mask, scores, B, T,
                                                                                   (double)kl_coef, out3);
    return launch_status();
}
