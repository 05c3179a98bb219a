// The whole path as one call (ppo_step) and its host-buffer variant (ppo_step_host): sequencing of the
// steps (the token-level ones fused into one launch that overlaps its neighbours) plus the host<->device copies.
#include "ppo_common.cuh"

#include <mutex>

using namespace ppo;

extern "C" int ppo_step(const ppo_step_io *io, int dtype, int32_t B, int32_t T, int64_t V, const ppo_params *p,
                        void *stream)
{
    if (!io || !p) return PPO_ERR_NULL;
    if (B <= 0 || T <= 0 || V <= 0) return PPO_ERR_SHAPE;
    if (!io->responses_out || !io->eos_index || !io->seq_len || !io->mask || !io->scores_out || !io->logprob ||
        !io->entropy || !io->ref_logprob || !io->kl || !io->rewards || !io->advantages || !io->returns ||
        !io->advantages_whitened || !io->workspace)
        return PPO_ERR_NULL;
    if (!io->responses || !io->scores || !io->values || !io->policy_logits || !io->ref_logits || !io->losses ||
        !io->dvalues)
        return PPO_ERR_NULL;
    if (p->eos_id == p->pad_id || !finite_f(p->kl_coef) || !finite_f(p->gamma) || !finite_f(p->lam) ||
        !(p->whiten_eps >= 0.f))
        return PPO_ERR_PARAM;
    if (reinterpret_cast<uintptr_t>(io->workspace) % 256) return PPO_ERR_ALIGN;
    const int64_t rows = (int64_t)B * T;
    if (rows >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // three launches: log-probs (policy and reference) -> [EOS trick + KL rewards + GAE, then loss
    // prologue + whitening in the last block] -> loss forward/backward.
    // Padding rows (after a sequence's first EOS) are masked out of every later step, so step 1 does not read
    // their logits: the log-prob kernel finds them from the sampled tokens alone and writes 0 there.
    int rc = PPO_ERR_UNSUPPORTED;
    if ((dtype == PPO_F32 || dtype == PPO_BF16) && V < ((int64_t)1 << 31) && p->temperature > 0.f &&
        finite_f(p->temperature) && option_value(PPO_OPT_ROW_ENGINE) != 2)
        rc = launch_logprob_pair(io->policy_logits, io->ref_logits, dtype, rows, (int)V, io->responses, nullptr, T,
                                 p->eos_id, kLog2e / p->temperature, io->logprob, io->entropy, io->ref_logprob,
                                 ws_header(io->workspace), true, s);
    const bool flags_cleared = rc == PPO_OK;
    if (rc == PPO_ERR_UNSUPPORTED) {   // layout without 16-byte packs (or the row engine was asked for): the EOS
                                       // trick first (for the mask), then one call per tensor
        rc = ppo_truncate_and_score(io->responses, B, T, p->eos_id, p->pad_id, io->scores, p->no_eos_score,
                                    io->responses_out, io->eos_index, io->seq_len, io->mask, io->scores_out, stream);
        if (rc) return rc;
        rc = ppo_logprob_entropy(io->policy_logits, dtype, rows, V, V, io->responses, io->mask, p->temperature,
                                 io->logprob, io->entropy, nullptr, io->workspace, stream);
        if (rc) return rc;
        rc = ppo_logprob_entropy(io->ref_logits, dtype, rows, V, V, io->responses, io->mask, p->temperature,
                                 io->ref_logprob, nullptr, nullptr, io->workspace, stream);
    }
    if (rc) return rc;
    rc = launch_rollout(io, B, T, p, flags_cleared, s);
    if (rc) return rc;
    return loss_fwd_bwd_prepared(io->loss_logits ? io->loss_logits : io->policy_logits, dtype, B, T, V, io->responses,
                                 io->mask, io->old_logprob ? io->old_logprob : io->logprob, io->advantages_whitened,
                                 io->values_new, io->values, io->returns, p, io->losses, io->dlogits, io->dvalues,
                                 io->new_logprob, io->new_entropy, io->dlogprob, io->workspace, stream, true);
}

namespace {

int copy_in(void *dst, const void *src, size_t bytes, cudaStream_t s)
{
    if (!src) return PPO_OK;          // optional input not supplied
    if (!dst) return PPO_ERR_NULL;    // supplied on the host but no staging buffer on the device
    PPO_RETURN_IF_CUDA(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, s));
    return PPO_OK;
}

// A [B, T, V] logits tensor: only the rows that ppo_step reads are copied - of each response the positions up to
// and including its first EOS (the EOS trick masks the rest out of every step; found here from the host's tokens).
// A response without EOS ends where the next one starts, so the two go out as one copy.
int copy_in_real_rows(void *dst, const void *src, const int32_t *responses, int32_t B, int32_t T, size_t row_bytes,
                      int32_t eos_id, cudaStream_t s)
{
    if (!src) return PPO_OK;
    if (!dst) return PPO_ERR_NULL;
    size_t run_off = 0, run_bytes = 0;   // copy being collected
    for (int32_t b = 0; b < B; ++b) {
        const int32_t *r = responses + (size_t)b * T;
        int32_t L = T;
        for (int32_t t = 0; t < T; ++t)
            if (r[t] == eos_id) { L = t + 1; break; }
        const size_t off = (size_t)b * T * row_bytes;
        if (run_bytes && run_off + run_bytes != off) {
            PPO_RETURN_IF_CUDA(cudaMemcpyAsync(static_cast<unsigned char *>(dst) + run_off,
                                               static_cast<const unsigned char *>(src) + run_off, run_bytes,
                                               cudaMemcpyHostToDevice, s));
            run_bytes = 0;
        }
        if (!run_bytes) run_off = off;
        run_bytes += (size_t)L * row_bytes;
    }
    if (run_bytes)
        PPO_RETURN_IF_CUDA(cudaMemcpyAsync(static_cast<unsigned char *>(dst) + run_off,
                                           static_cast<const unsigned char *>(src) + run_off, run_bytes,
                                           cudaMemcpyHostToDevice, s));
    return PPO_OK;
}

// Second copy queue of ppo_step_host. One queue leaves the link idle between two copies (about 4 us per copy, 8% of
// the transfer time at 128 copies of 2.5 MB); with the policy tensor on the caller's stream and the reference tensor
// on a side stream the gaps of one queue are filled by the other. One side stream and two events per device, created
// on the first call on that device and kept until the process exits.
struct CopyLane {
    cudaStream_t side = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};
std::mutex g_lane_mutex;   // held while a call enqueues its fork / join, so that two host threads cannot interleave them

int copy_lane(CopyLane **out)
{
    static CopyLane lanes[64];
    int dev = 0;
    PPO_RETURN_IF_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PPO_ERR_UNSUPPORTED;
    CopyLane &l = lanes[dev];
    if (!l.side) {
        cudaStream_t st = nullptr;
        PPO_RETURN_IF_CUDA(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
        PPO_RETURN_IF_CUDA(cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming));
        PPO_RETURN_IF_CUDA(cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming));
        l.side = st;
    }
    *out = &l;
    return PPO_OK;
}

int copy_out(void *dst, const void *src, size_t bytes, cudaStream_t s)
{
    if (!dst) return PPO_OK;          // the caller does not want this output on the host
    if (!src) return PPO_ERR_NULL;
    PPO_RETURN_IF_CUDA(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, s));
    return PPO_OK;
}

}   // namespace

#define PPO_TRY(expr)          \
    do {                       \
        int rc__ = (expr);     \
        if (rc__) return rc__; \
    } while (0)

extern "C" int ppo_step_host(const ppo_step_io *host, const ppo_step_io *dev, int dtype, int32_t B, int32_t T,
                             int64_t V, const ppo_params *p, void *stream)
{
    if (!host || !dev || !p) return PPO_ERR_NULL;
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (B <= 0 || T <= 0 || V <= 0) return PPO_ERR_SHAPE;
    if (!host->policy_logits || !host->ref_logits || !host->responses || !host->scores || !host->values ||
        !host->values_new)
        return PPO_ERR_NULL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t bt = (size_t)B * (size_t)T, es = dtype == PPO_F32 ? 4 : 2;
    const size_t logits_bytes = bt * (size_t)V * es;
    // device staging buffers are written here, so drop the const the struct carries for inputs
    {
        // the reference tensor goes through the side queue, everything else through the caller's stream; the side
        // queue starts after the work already in the stream (which may still read the staging buffers) and the
        // stream continues after the side queue's last copy
        std::lock_guard<std::mutex> guard(g_lane_mutex);
        CopyLane *lane = nullptr;
        PPO_TRY(copy_lane(&lane));
        PPO_RETURN_IF_CUDA(cudaEventRecord(lane->fork, s));
        PPO_RETURN_IF_CUDA(cudaStreamWaitEvent(lane->side, lane->fork, 0));
        PPO_TRY(copy_in_real_rows(const_cast<void *>(dev->ref_logits), host->ref_logits, host->responses, B, T,
                                  (size_t)V * es, p->eos_id, lane->side));
        PPO_RETURN_IF_CUDA(cudaEventRecord(lane->join, lane->side));
        PPO_TRY(copy_in_real_rows(const_cast<void *>(dev->policy_logits), host->policy_logits, host->responses, B, T,
                                  (size_t)V * es, p->eos_id, s));
        PPO_TRY(copy_in_real_rows(const_cast<void *>(dev->loss_logits), host->loss_logits, host->responses, B, T,
                                  (size_t)V * es, p->eos_id, s));
        PPO_RETURN_IF_CUDA(cudaStreamWaitEvent(s, lane->join, 0));
    }
    PPO_TRY(copy_in(const_cast<int32_t *>(dev->responses), host->responses, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->scores), host->scores, (size_t)B * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->values), host->values, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->values_new), host->values_new, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->old_logprob), host->old_logprob, bt * 4, s));
    ppo_step_io run = *dev;
    if (!host->loss_logits) run.loss_logits = nullptr;
    if (!host->old_logprob) run.old_logprob = nullptr;
    PPO_TRY(ppo_step(&run, dtype, B, T, V, p, stream));
    PPO_TRY(copy_out(host->responses_out, dev->responses_out, bt * 4, s));
    PPO_TRY(copy_out(host->eos_index, dev->eos_index, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->seq_len, dev->seq_len, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->mask, dev->mask, bt, s));
    PPO_TRY(copy_out(host->scores_out, dev->scores_out, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->logprob, dev->logprob, bt * 4, s));
    PPO_TRY(copy_out(host->entropy, dev->entropy, bt * 4, s));
    PPO_TRY(copy_out(host->ref_logprob, dev->ref_logprob, bt * 4, s));
    PPO_TRY(copy_out(host->kl, dev->kl, bt * 4, s));
    PPO_TRY(copy_out(host->rewards, dev->rewards, bt * 4, s));
    PPO_TRY(copy_out(host->advantages, dev->advantages, bt * 4, s));
    PPO_TRY(copy_out(host->returns, dev->returns, bt * 4, s));
    PPO_TRY(copy_out(host->advantages_whitened, dev->advantages_whitened, bt * 4, s));
    PPO_TRY(copy_out(host->whiten_stats, dev->whiten_stats, 3 * 4, s));
    PPO_TRY(copy_out(host->losses, dev->losses, 8 * 4, s));
    PPO_TRY(copy_out(host->dlogits, dev->dlogits, logits_bytes, s));
    PPO_TRY(copy_out(host->dvalues, dev->dvalues, bt * 4, s));
    PPO_TRY(copy_out(host->new_logprob, dev->new_logprob, bt * 4, s));
    PPO_TRY(copy_out(host->new_entropy, dev->new_entropy, bt * 4, s));
    PPO_TRY(copy_out(host->dlogprob, dev->dlogprob, bt * 4, s));
    PPO_RETURN_IF_CUDA(cudaStreamSynchronize(s));
    return PPO_OK;
}


// ---------------------------------------------------------------- the fused-LM-head config as one call
extern "C" int ppo_lmhead_step(const ppo_lmhead_step_io *io, int32_t B, int32_t T, int64_t K, int64_t V,
                               const ppo_params *p, void *stream)
{
    if (!io || !p) return PPO_ERR_NULL;
    if (B <= 0 || T <= 0 || K <= 0 || V <= 0) return PPO_ERR_SHAPE;
    if (!io->H || !io->W || !io->W_ref || !io->responses || !io->scores || !io->values || !io->values_new)
        return PPO_ERR_NULL;
    if (!io->responses_out || !io->eos_index || !io->seq_len || !io->mask || !io->scores_out || !io->logprob ||
        !io->entropy || !io->ref_logprob || !io->kl || !io->rewards || !io->advantages || !io->returns ||
        !io->advantages_whitened || !io->losses || !io->dvalues || !io->workspace)
        return PPO_ERR_NULL;
    const int64_t M = (int64_t)B * T;
    PPO_TRY(ppo_truncate_and_score(io->responses, B, T, p->eos_id, p->pad_id, io->scores, p->no_eos_score,
                                   io->responses_out, io->eos_index, io->seq_len, io->mask, io->scores_out, stream));
    PPO_TRY(ppo_lmhead_logprob_entropy(io->H, io->W, M, K, V, io->responses, io->mask, p->temperature, io->logprob,
                                       io->entropy, io->lse, io->workspace, stream));
    PPO_TRY(ppo_lmhead_logprob_entropy(io->H, io->W_ref, M, K, V, io->responses, io->mask, p->temperature,
                                       io->ref_logprob, nullptr, nullptr, io->workspace, stream));
    PPO_TRY(ppo_kl_rewards(io->logprob, io->ref_logprob, io->mask, io->seq_len, io->scores_out, B, T, p->kl_coef,
                           io->kl, io->rewards, stream));
    if (p->whiten_rewards)   // optional reward whitening: mean kept, in place, before GAE
        PPO_TRY(ppo_whiten(io->rewards, io->mask, M, 0, p->whiten_eps, io->rewards, nullptr, io->workspace, stream));
    PPO_TRY(ppo_gae(io->rewards, io->values, io->seq_len, B, T, p->gamma, p->lam, io->advantages, io->returns, stream));
    PPO_TRY(ppo_whiten(io->advantages, io->mask, M, 1, p->whiten_eps, io->advantages_whitened, io->whiten_stats,
                       io->workspace, stream));
    return ppo_loss_from_logprob(io->logprob, io->entropy, B, T, io->mask, io->old_logprob ? io->old_logprob : io->logprob,
                                 io->advantages_whitened, io->values_new, io->values, io->returns, p, io->losses,
                                 io->dlogprob, io->dvalues, io->workspace, stream);
}

extern "C" int ppo_lmhead_step_host(const ppo_lmhead_step_io *host, const ppo_lmhead_step_io *dev, int32_t B, int32_t T,
                                    int64_t K, int64_t V, const ppo_params *p, void *stream)
{
    if (!host || !dev || !p) return PPO_ERR_NULL;
    if (B <= 0 || T <= 0 || K <= 0 || V <= 0) return PPO_ERR_SHAPE;
    if (!host->H || !host->W || !host->W_ref || !host->responses || !host->scores || !host->values || !host->values_new)
        return PPO_ERR_NULL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t bt = (size_t)B * (size_t)T, w_bytes = (size_t)K * (size_t)V * 2;
    // (the rows of H behind a response's first EOS are never multiplied: they are not copied either)
    PPO_TRY(copy_in_real_rows(const_cast<void *>(dev->H), host->H, host->responses, B, T, (size_t)K * 2, p->eos_id, s));
    PPO_TRY(copy_in(const_cast<void *>(dev->W), host->W, w_bytes, s));
    PPO_TRY(copy_in(const_cast<void *>(dev->W_ref), host->W_ref, w_bytes, s));
    PPO_TRY(copy_in(const_cast<int32_t *>(dev->responses), host->responses, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->scores), host->scores, (size_t)B * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->values), host->values, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->values_new), host->values_new, bt * 4, s));
    PPO_TRY(copy_in(const_cast<float *>(dev->old_logprob), host->old_logprob, bt * 4, s));
    ppo_lmhead_step_io run = *dev;
    if (!host->old_logprob) run.old_logprob = nullptr;
    PPO_TRY(ppo_lmhead_step(&run, B, T, K, V, p, stream));
    PPO_TRY(copy_out(host->responses_out, dev->responses_out, bt * 4, s));
    PPO_TRY(copy_out(host->eos_index, dev->eos_index, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->seq_len, dev->seq_len, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->mask, dev->mask, bt, s));
    PPO_TRY(copy_out(host->scores_out, dev->scores_out, (size_t)B * 4, s));
    PPO_TRY(copy_out(host->logprob, dev->logprob, bt * 4, s));
    PPO_TRY(copy_out(host->entropy, dev->entropy, bt * 4, s));
    PPO_TRY(copy_out(host->lse, dev->lse, bt * 4, s));
    PPO_TRY(copy_out(host->ref_logprob, dev->ref_logprob, bt * 4, s));
    PPO_TRY(copy_out(host->kl, dev->kl, bt * 4, s));
    PPO_TRY(copy_out(host->rewards, dev->rewards, bt * 4, s));
    PPO_TRY(copy_out(host->advantages, dev->advantages, bt * 4, s));
    PPO_TRY(copy_out(host->returns, dev->returns, bt * 4, s));
    PPO_TRY(copy_out(host->advantages_whitened, dev->advantages_whitened, bt * 4, s));
    PPO_TRY(copy_out(host->whiten_stats, dev->whiten_stats, 3 * 4, s));
    PPO_TRY(copy_out(host->losses, dev->losses, 8 * 4, s));
    PPO_TRY(copy_out(host->dlogprob, dev->dlogprob, bt * 4, s));
    PPO_TRY(copy_out(host->dvalues, dev->dvalues, bt * 4, s));
    PPO_RETURN_IF_CUDA(cudaStreamSynchronize(s));
    return PPO_OK;
}
