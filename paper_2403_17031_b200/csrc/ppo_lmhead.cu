// Step 7: LM-head GEMM fused with the log-prob / entropy reduction (placeholder translation
// unit; the tcgen05 kernel is added separately).
#include "ppo_common.cuh"

using namespace ppo;

extern "C" size_t ppo_lmhead_workspace_bytes(int64_t M, int64_t K, int64_t V)
{
    (void)K;
    (void)V;
    if (M <= 0) return kHeaderBytes;
    return kHeaderBytes + align256((size_t)M * 64);
}

extern "C" int ppo_lmhead_logprob_entropy(const void *H, const void *W, int64_t M, int64_t K, int64_t V,
                                          const int32_t *tokens, const uint8_t *mask, float temperature,
                                          float *logprob, float *entropy, float *lse, void *workspace,
                                          void *stream)
{
    (void)H; (void)W; (void)M; (void)K; (void)V; (void)tokens; (void)mask; (void)temperature;
    (void)logprob; (void)entropy; (void)lse; (void)workspace; (void)stream;
    return PPO_ERR_UNSUPPORTED;
}
