// Token-level kernels: everything that touches only [B,T]-sized arrays (steps 2-5, the loss
// reductions, workspace and status plumbing). These move <0.1% of the path's bytes and are
// bound by launch latency; each is a single small launch.
#include "ppo_common.cuh"

namespace ppo {

static int g_options[8] = {0, 0, 0, 0, 0, 0, 0, 0};
int option_value(int key) { return (key >= 0 && key < 8) ? g_options[key] : 0; }

// ---------------------------------------------------------------- step 2: EOS trick
// One warp per response: lanes stride over t, a warp-wide min finds the first EOS.
__device__ __forceinline__ int truncate_sequence(const int32_t *responses, int b, int T, int eos_id, int pad_id,
                                                  const float *__restrict__ scores, float no_eos_score,
                                                  int32_t *responses_out, int32_t *__restrict__ eos_index,
                                                  int32_t *__restrict__ seq_len, uint8_t *__restrict__ mask,
                                                  float *__restrict__ scores_out, int lane)
{
    const int32_t *r = responses + (int64_t)b * T;
    int first = T;
    for (int t = lane; t < T; t += 32)
        if (r[t] == eos_id) { first = t; break; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, off));
    const int e = first < T ? first : -1;
    const int L = first < T ? first + 1 : T;
    for (int t = lane; t < T; t += 32) {
        const int64_t i = (int64_t)b * T + t;
        const int32_t tok = r[t];
        if (responses_out) responses_out[i] = t < L ? tok : pad_id;
        if (mask) mask[i] = (uint8_t)(t < L);
    }
    if (lane == 0) {
        if (eos_index) eos_index[b] = e;
        if (seq_len) seq_len[b] = L;
        if (scores_out) scores_out[b] = e >= 0 ? scores[b] : no_eos_score;
    }
    return L;   // known to every lane
}

__global__ void __launch_bounds__(128)
truncate_kernel(const int32_t *responses, int B, int T, int eos_id, int pad_id,
                const float *__restrict__ scores, float no_eos_score, int32_t *responses_out,
                int32_t *__restrict__ eos_index, int32_t *__restrict__ seq_len, uint8_t *__restrict__ mask,
                float *__restrict__ scores_out)
{
    const int b = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (b >= B) return;
    truncate_sequence(responses, b, T, eos_id, pad_id, scores, no_eos_score, responses_out, eos_index, seq_len, mask,
                      scores_out, threadIdx.x & 31);
}

// ---------------------------------------------------------------- step 3: KL rewards
// Explicitly rounded fp32 operations: the fused kernel below must reproduce these bits.
__device__ __forceinline__ float kl_reward(float k, bool real, float kl_coef, bool last, float score)
{
    float r = real ? __fmul_rn(-kl_coef, k) : 0.f;
    if (last) r = __fadd_rn(r, score);
    return r;
}

__global__ void __launch_bounds__(256)
kl_rewards_kernel(const float *__restrict__ logprob, const float *__restrict__ ref_logprob,
                  const uint8_t *__restrict__ mask, const int32_t *__restrict__ seq_len,
                  const float *__restrict__ scores, int B, int T, float kl_coef, float *__restrict__ kl,
                  float *__restrict__ rewards)
{
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= (int64_t)B * T) return;
    const int b = (int)(i / T), t = (int)(i - (int64_t)b * T);
    const bool real = mask[i] != 0;
    const float k = real ? __fsub_rn(logprob[i], ref_logprob[i]) : 0.f;
    if (kl) kl[i] = k;
    if (rewards) rewards[i] = kl_reward(k, real, kl_coef, t == seq_len[b] - 1, scores[b]);
}

// ---------------------------------------------------------------- step 4: GAE
// One warp per sequence. Lane l owns the contiguous time segment [l*S, (l+1)*S); running the
// recurrence A_t = delta_t + c*A_{t+1} over a segment is an affine map of the incoming A, so
// (1) each lane folds its segment into (a, b), (2) a reverse inclusive warp scan composes the
// maps, (3) each lane replays its segment from the correct incoming value. fp64 throughout.
// `reward(t)` yields the fp32 reward of token t.
template <typename RewardFn>
__device__ __forceinline__ void gae_sequence(RewardFn reward, const float *__restrict__ v, int L, int T, double gamma,
                                             double c, float *__restrict__ advantages, float *__restrict__ returns,
                                             int lane)
{
    L = L < 0 ? 0 : (L > T ? T : L);
    const int S = (T + 31) / 32;
    const int s0 = min(lane * S, T), s1 = min(s0 + S, T);
    double a = 1.0, bb = 0.0;
    for (int t = s1 - 1; t >= s0; --t) {
        double d = 0.0;
        if (t < L) {
            const double vn = (t + 1 < L) ? (double)v[t + 1] : 0.0;
            d = ((double)reward(t) + gamma * vn) - (double)v[t];
        }
        bb = d + c * bb;
        a = c * a;
    }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double aj = __shfl_down_sync(0xffffffffu, a, off);
        const double bj = __shfl_down_sync(0xffffffffu, bb, off);
        if (lane + off < 32) {
            bb = bb + a * bj;
            a = a * aj;
        }
    }
    double A = __shfl_down_sync(0xffffffffu, bb, 1);
    if (lane == 31) A = 0.0;
    for (int t = s1 - 1; t >= s0; --t) {
        if (t < L) {
            const double vn = (t + 1 < L) ? (double)v[t + 1] : 0.0;
            const double d = ((double)reward(t) + gamma * vn) - (double)v[t];
            A = d + c * A;
            advantages[t] = (float)A;
            returns[t] = (float)(A + (double)v[t]);
        } else {
            A = c * A;
            advantages[t] = 0.f;
            returns[t] = 0.f;
        }
    }
}

__global__ void __launch_bounds__(128)
gae_kernel(const float *__restrict__ rewards, const float *__restrict__ values,
           const int32_t *__restrict__ seq_len, int B, int T, double gamma, double c /* gamma*lam */,
           float *__restrict__ advantages, float *__restrict__ returns)
{
    const int b = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (b >= B) return;
    const float *r = rewards + (int64_t)b * T;
    gae_sequence([r](int t) { return r[t]; }, values + (int64_t)b * T, seq_len[b], T, gamma, c,
                 advantages + (int64_t)b * T, returns + (int64_t)b * T, threadIdx.x & 31);
}

// ---------------------------------------------------------------- step 5: masked whitening
// One block: three passes over the (L1/L2-resident) array, fp64 sums in a fixed order.
constexpr int kWhitenThreads = 1024;
__device__ __forceinline__ void whiten_block(const float *x, const uint8_t *__restrict__ mask, int64_t n_elems,
                                             int shift_mean, float eps, float *out, float *__restrict__ stats3,
                                             int *status, double *red /* 32 doubles */)
{
    double sum = 0.0, cnt = 0.0;
    for (int64_t i = threadIdx.x; i < n_elems; i += kWhitenThreads)
        if (!mask || mask[i]) { sum += (double)x[i]; cnt += 1.0; }
    sum = block_sum<kWhitenThreads>(sum, red);
    cnt = block_sum<kWhitenThreads>(cnt, red);
    const double mean = cnt > 0.0 ? sum / cnt : 0.0;
    double ss = 0.0;
    for (int64_t i = threadIdx.x; i < n_elems; i += kWhitenThreads)
        if (!mask || mask[i]) { const double d = (double)x[i] - mean; ss += d * d; }
    ss = block_sum<kWhitenThreads>(ss, red);
    const double var = cnt > 0.0 ? ss / cnt : 0.0;
    const double inv = 1.0 / sqrt(var + (double)eps);
    const double back = shift_mean ? 0.0 : mean;
    for (int64_t i = threadIdx.x; i < n_elems; i += kWhitenThreads) {
        float y = 0.f;
        if (!mask || mask[i]) y = (float)(((double)x[i] - mean) * inv + back);
        out[i] = y;
    }
    if (threadIdx.x == 0) {
        if (stats3) { stats3[0] = (float)mean; stats3[1] = (float)var; stats3[2] = (float)cnt; }
        if (cnt == 0.0 && status) atomicOr(status, PPO_DEV_EMPTY_MASK);
    }
}

__global__ void __launch_bounds__(kWhitenThreads)
whiten_kernel(const float *x, const uint8_t *__restrict__ mask, int64_t n_elems, int shift_mean, float eps,
              float *out, float *__restrict__ stats3, int *status)
{
    __shared__ double red[32];
    whiten_block(x, mask, n_elems, shift_mean, eps, out, stats3, status, red);
}

// ---------------------------------------------------------------- loss plumbing
constexpr int kReduceThreads = 1024;

// Prologue of a loss call (one block): counts the real tokens, resets the work counters and writes
// the row order: indices of real rows ascending from the front, masked rows from the back. Each
// thread owns one contiguous segment of rows, so the order is deterministic.
__device__ __forceinline__ void loss_prepare_block(const uint8_t *mask, int64_t rows, WorkspaceHeader *hdr,
                                                   int32_t *__restrict__ order, int *warp_tot /* 32 ints */,
                                                   bool publish /* a loss kernel may be waiting for the result */,
                                                   bool flag_empty = true /* no row with mask 1: status bit */)
{
    // segments are multiples of 16 rows so that a 16-byte aligned mask is read 16 rows per load (the result does
    // not depend on the segment length: segments are contiguous and ascending)
    const bool vec = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
    int64_t seg = (rows + kReduceThreads - 1) / kReduceThreads;
    if (vec) seg = (seg + 15) & ~(int64_t)15;
    const int64_t r0 = min(rows, (int64_t)threadIdx.x * seg), r1 = min(rows, r0 + seg);
    const int64_t rv = vec ? r0 + ((r1 - r0) & ~(int64_t)15) : r0;   // [r0, rv): whole groups of 16 rows
    int c = 0;
#pragma unroll 4
    for (int64_t r = r0; r < rv; r += 16) {
        const uint4 v = *reinterpret_cast<const uint4 *>(mask + r);
        c += (__popc(__vcmpne4(v.x, 0u)) + __popc(__vcmpne4(v.y, 0u)) + __popc(__vcmpne4(v.z, 0u)) +
              __popc(__vcmpne4(v.w, 0u))) >> 3;
    }
    for (int64_t r = rv; r < r1; ++r) c += mask[r] ? 1 : 0;
    // block exclusive scan of c
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = c;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane], wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off) wi += t;
        }
        warp_tot[lane] = wi - w;   // exclusive prefix of the warp totals
        if (lane == 31) {
            hdr->n_tokens = wi;
            hdr->masked_next = 0;
            hdr->masked_tail = 0;
            hdr->real_next = 0;
            hdr->done_blocks = 0;
            hdr->order_sig[0] = (unsigned long long)reinterpret_cast<uintptr_t>(mask);
            hdr->order_sig[1] = (unsigned long long)rows;
            hdr->order_sig[2] = (unsigned long long)reinterpret_cast<uintptr_t>(order);
            if (wi == 0 && flag_empty) atomicOr(&hdr->status, PPO_DEV_EMPTY_MASK);
        }
    }
    __syncthreads();
    int real_pos = warp_tot[warp] + incl - c;            // real rows before this segment
    int64_t masked_pos = r0 - real_pos;                   // masked rows before this segment
    for (int64_t r = r0; r < rv; r += 16) {
        const uint4 v = *reinterpret_cast<const uint4 *>(mask + r);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            if ((w[q >> 2] >> ((q & 3) * 8)) & 0xffu) order[real_pos++] = (int32_t)(r + q);
            else order[rows - 1 - masked_pos++] = (int32_t)(r + q);
        }
    }
    for (int64_t r = rv; r < r1; ++r) {
        if (mask[r]) order[real_pos++] = (int32_t)r;
        else order[rows - 1 - masked_pos++] = (int32_t)r;
    }
    if (!publish) return;
    __syncthreads();
    // a loss kernel that is already running may go on; the flag carries the token count (+1) it needs first
    if (threadIdx.x == 0) flag_set(&hdr->order_ready, *reinterpret_cast<volatile int *>(&hdr->n_tokens) + 1, kFlagOrder);
}

__global__ void __launch_bounds__(kReduceThreads)
loss_prepare_kernel(const uint8_t *__restrict__ mask, int64_t rows, WorkspaceHeader *hdr, int32_t *__restrict__ order,
                    int flag_empty)
{
    __shared__ int warp_tot[32];
    // the loss kernel that follows is launched as a programmatic dependent: it may start now and waits on the
    // two flags, which are cleared before this (only) block lets it launch
    if (threadIdx.x == 0) {
        hdr->order_ready = 0;
        hdr->adv_ready = 0;
        __threadfence();
    }
    __syncthreads();
    grid_dependents_may_launch();
    loss_prepare_block(mask, rows, hdr, order, warp_tot, true, flag_empty != 0);
    if (threadIdx.x == 0) flag_set(&hdr->adv_ready, 1, kFlagAdv);   // stand-alone loss call: its other inputs exist already
}

// ---------------------------------------------------------------- fused launch of ppo_step
// Everything token-level in one launch, after the log-prob launch (which finds the padding rows by itself):
// one warp per sequence runs the EOS trick, the KL rewards and GAE; one extra block runs the loss
// prologue (token count, row order) as soon as every sequence has had the EOS trick, and the last
// sequence block to finish whitens the advantages of the whole batch - each with exactly the code and
// thread assignment of the stand-alone kernels, so the results are bit-identical to calling the steps
// one by one. The launch overlaps its neighbours (see grid_dependency_wait / flag_set below).
//
// PHASE 0: all of it. With reward whitening (detail "(Optional) Reward whitening": the rewards of the
// batch are whitened without shifting the mean BEFORE GAE) the advantages need batch-wide statistics of
// the rewards first, so the work is split over two launches of the same kernel:
// PHASE 1: EOS trick + KL rewards; the last block whitens the rewards in place (shift_mean = 0);
// PHASE 2: GAE on the rewards array; the last block runs the loss prologue + advantage whitening.
template <int PHASE>
__global__ void __launch_bounds__(kWhitenThreads)
rollout_kernel(const int32_t *responses, int B, int T, int eos_id, int pad_id, const float *__restrict__ scores,
               float no_eos_score, int32_t *responses_out, int32_t *eos_index, int32_t *seq_len, uint8_t *mask,
               float *__restrict__ scores_out, const float *__restrict__ logprob,
               const float *__restrict__ ref_logprob, const float *__restrict__ values, float kl_coef, double gamma,
               double c, float eps, float *__restrict__ kl, float *rewards, float *advantages,
               float *__restrict__ returns, float *whitened, float *__restrict__ stats3, WorkspaceHeader *hdr,
               int32_t *__restrict__ order, int clear_flags)
{
    static_assert(kWhitenThreads == kReduceThreads, "one block shape for both block-wide helpers");
    __shared__ double red[32];
    __shared__ int warp_tot[32];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * (kWhitenThreads / 32) + (threadIdx.x >> 5);
    const int64_t rows = (int64_t)B * T;
    // The loss kernel of this step may start while this kernel runs (launch_dependent) and waits on the two
    // flags. They are 0 by now: cleared by the launch before this one, or here before any block lets the loss
    // kernel launch (it launches once ALL blocks have said so).
    if (clear_flags) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            hdr->order_ready = 0;
            hdr->adv_ready = 0;
            __threadfence();
        }
        __syncthreads();
    }
    if (PHASE == 0) grid_dependents_may_launch();
    // This kernel itself may have been scheduled while the log-prob kernel before it was draining. The EOS trick
    // and the loss prologue need the sampled tokens only (an input that nothing writes), so in PHASE 0 they run
    // before the wait for that kernel; everything that reads log-probs comes after it.
    if (PHASE != 0) grid_dependency_wait();

    // tickets: the block that draws the last one continues with the batch-wide step
    const auto last_block = [&](int *counter, int n_blocks) {
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const int ticket = atomicAdd(counter, 1);
            is_last = ticket == n_blocks - 1;
            if (is_last) *counter = 0;   // ready for the next call
        }
        __syncthreads();
        const bool last = is_last != 0;
        if (last) __threadfence();
        return last;
    };

    if (PHASE == 2) {
        if (b < B) {
            const float *r = rewards + (int64_t)b * T;
            gae_sequence([r](int t) { return r[t]; }, values + (int64_t)b * T, seq_len[b], T, gamma, c,
                         advantages + (int64_t)b * T, returns + (int64_t)b * T, lane);
        }
        if (!last_block(&hdr->step_blocks, (int)gridDim.x)) return;
        loss_prepare_block(mask, rows, hdr, order, warp_tot, true);
        __syncthreads();
        whiten_block(advantages, mask, rows, 1, eps, whitened, stats3, &hdr->status, red);
        __syncthreads();
        if (threadIdx.x == 0) flag_set(&hdr->adv_ready, 1, kFlagAdv);
        return;
    }

    // PHASE 0 has one block more than the sequences need: it waits until every other block has done the EOS
    // trick (the mask is all the loss prologue needs), then writes token count and row order and publishes
    // them, while the other blocks go on with rewards and advantages.
    const int n_seq_blocks = PHASE == 0 ? (int)gridDim.x - 1 : (int)gridDim.x;
    if (PHASE == 0 && (int)blockIdx.x == n_seq_blocks) {
        if (threadIdx.x == 0) {
            bool done = false;
            for (uint32_t it = 0; it < (1u << 20) && !done; ++it) {
                int v;
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(&hdr->step_blocks) : "memory");
                done = v >= n_seq_blocks;
                if (!done) __nanosleep(100);
            }
            if (!done) atomicOr(&hdr->status, PPO_DEV_TIMEOUT);
            hdr->step_blocks = 0;   // ready for the next call
        }
        __syncthreads();
        loss_prepare_block(mask, rows, hdr, order, warp_tot, true);
        return;
    }
    int L = 0;
    if (b < B)
        L = truncate_sequence(responses, b, T, eos_id, pad_id, scores, no_eos_score, responses_out, eos_index, seq_len,
                              mask, scores_out, lane);
    if (PHASE == 0) {   // tell the prologue block, then wait for the log-probs
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) atomicAdd(&hdr->step_blocks, 1);
        grid_dependency_wait();
    }
    if (b < B) {
        int first_eos = 0;   // whether the sequence has an EOS decides the score that is used
        {
            const int32_t *r = responses + (int64_t)b * T;
            first_eos = (L < T) || (r[T - 1] == eos_id);
        }
        const float score = first_eos ? scores[b] : no_eos_score;
        const float *lp = logprob + (int64_t)b * T, *lr = ref_logprob + (int64_t)b * T;
        for (int t = lane; t < T; t += 32) {
            const bool real = t < L;
            const float k = real ? __fsub_rn(lp[t], lr[t]) : 0.f;
            kl[(int64_t)b * T + t] = k;
            rewards[(int64_t)b * T + t] = kl_reward(k, real, kl_coef, t == L - 1, score);
        }
        if (PHASE == 0)
            gae_sequence(
                [=](int t) {
                    return kl_reward(t < L ? __fsub_rn(lp[t], lr[t]) : 0.f, t < L, kl_coef, t == L - 1, score);
                },
                values + (int64_t)b * T, L, T, gamma, c, advantages + (int64_t)b * T, returns + (int64_t)b * T, lane);
    }
    if (!last_block(PHASE == 0 ? &hdr->step_blocks2 : &hdr->step_blocks, n_seq_blocks)) return;
    if (PHASE == 1) {
        whiten_block(rewards, mask, rows, 0, eps, rewards, nullptr, &hdr->status, red);
        return;
    }
    whiten_block(advantages, mask, rows, 1, eps, whitened, stats3, &hdr->status, red);
    __syncthreads();
    if (threadIdx.x == 0) flag_set(&hdr->adv_ready, 1, kFlagAdv);
}

// Sum the per-token partials (fixed thread assignment, fp64) and write the eight loss scalars.
__global__ void __launch_bounds__(kReduceThreads)
loss_finalize_kernel(const float *__restrict__ partials, int64_t rows, const WorkspaceHeader *hdr, float vf_coef,
                     float *__restrict__ losses)
{
    __shared__ double red[6 * 32];
    reduce_loss_partials<kReduceThreads>(partials, rows, hdr->n_tokens, vf_coef, losses, red, (int)threadIdx.x,
                                         [] { __syncthreads(); });
}

// Step 6 at log-prob level (the logits were never materialised): one thread per token.
__global__ void __launch_bounds__(256)
loss_from_logprob_kernel(const float *__restrict__ new_logprob, const float *__restrict__ entropy, int64_t rows,
                         const uint8_t *__restrict__ mask, const float *__restrict__ old_logprob,
                         const float *__restrict__ advantages, const float *__restrict__ values_new,
                         const float *__restrict__ values_old, const float *__restrict__ returns, float eps,
                         float eps_v, float c1, const WorkspaceHeader *hdr, float *__restrict__ partials,
                         float *__restrict__ dlogprob, float *__restrict__ dvalues)
{
    const int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (r >= rows) return;
    float4 p0 = make_float4(0.f, 0.f, 0.f, 0.f), p1 = make_float4(0.f, 0.f, 0.f, 0.f);
    float g = 0.f, dv = 0.f;
    if (mask[r]) {
        const TokenLoss tl = token_loss(new_logprob[r], old_logprob[r], advantages[r], values_new[r],
                                        values_old[r], returns[r], eps, eps_v, c1, (double)hdr->n_tokens);
        p0 = make_float4(tl.pg, tl.vf, tl.kl, tl.pg_clipped);
        p1 = make_float4(tl.vf_clipped, entropy ? entropy[r] : 0.f, 0.f, 0.f);
        g = tl.g;
        dv = tl.dvalue;
    }
    reinterpret_cast<float4 *>(partials + r * kPartialsPerToken)[0] = p0;
    reinterpret_cast<float4 *>(partials + r * kPartialsPerToken)[1] = p1;
    if (dlogprob) dlogprob[r] = g;
    dvalues[r] = dv;
}

int launch_loss_prepare(const uint8_t *mask, int64_t rows, void *workspace, cudaStream_t s)
{
    loss_prepare_kernel<<<1, kReduceThreads, 0, s>>>(mask, rows, ws_header(workspace), ws_order(workspace, rows), 1);
    return launch_status();
}

int launch_row_order(const uint8_t *mask, int64_t rows, WorkspaceHeader *hdr, int32_t *order, cudaStream_t s)
{
    // (an empty selection is not an error for the caller of this one: no status bit)
    loss_prepare_kernel<<<1, kReduceThreads, 0, s>>>(mask, rows, hdr, order, 0);
    return launch_status();
}

int launch_rollout(const ppo_step_io *io, int B, int T, const ppo_params *p, bool flags_cleared, cudaStream_t s)
{
    const unsigned nb = (unsigned)((B + kWhitenThreads / 32 - 1) / (kWhitenThreads / 32));
#define PPO_LAUNCH_ROLLOUT(PHASE, GRID, CLEAR)                                                                       \
    launch_dependent(rollout_kernel<PHASE>, dim3(GRID), dim3(kWhitenThreads), 0, s,                                  \
        io->responses, B, T, p->eos_id, p->pad_id, io->scores, p->no_eos_score, io->responses_out, io->eos_index,    \
        io->seq_len, io->mask, io->scores_out, io->logprob, io->ref_logprob, io->values, p->kl_coef,                 \
        (double)p->gamma, (double)p->gamma * (double)p->lam, p->whiten_eps, io->kl, io->rewards, io->advantages,     \
        io->returns, io->advantages_whitened, io->whiten_stats, ws_header(io->workspace),                            \
        ws_order(io->workspace, (int64_t)B * T), CLEAR)
    if (p->whiten_rewards) {
        PPO_LAUNCH_ROLLOUT(1, nb, flags_cleared ? 0 : 1);
        PPO_LAUNCH_ROLLOUT(2, nb, 0);
    } else {
        PPO_LAUNCH_ROLLOUT(0, nb + 1, flags_cleared ? 0 : 1);   // + the block that runs the loss prologue
    }
#undef PPO_LAUNCH_ROLLOUT
    return launch_status();
}

int launch_loss_finalize(int64_t rows, float vf_coef, float *losses, void *workspace, cudaStream_t s)
{
    loss_finalize_kernel<<<1, kReduceThreads, 0, s>>>(ws_partials(workspace), rows, ws_header(workspace), vf_coef,
                                                      losses);
    return launch_status();
}

}   // namespace ppo

using namespace ppo;

extern "C" void ppo_default_params(ppo_params *p)
{
    if (!p) return;
    p->temperature = 0.7f;
    p->kl_coef = 0.05f;
    p->gamma = 1.0f;
    p->lam = 0.95f;
    p->cliprange = 0.2f;
    p->cliprange_value = 0.2f;
    p->vf_coef = 0.1f;
    p->no_eos_score = -1.0f;
    p->whiten_eps = 1e-8f;
    p->eos_id = 0;
    p->pad_id = 1;
    p->whiten_rewards = 0;
}

extern "C" int ppo_version(void) { return 100; }

extern "C" int ppo_set_option(int key, int value)
{
    if ((key == PPO_OPT_LOSS_ROW_CACHE && value >= 0 && value <= 2) ||
        (key == PPO_OPT_ROW_ENGINE && value >= 0 && value <= 2)) {
        g_options[key] = value;
        return PPO_OK;
    }
    return PPO_ERR_PARAM;
}

extern "C" size_t ppo_workspace_bytes(int32_t B, int32_t T, int64_t V)
{
    (void)V;
    if (B <= 0 || T <= 0) return kHeaderBytes;
    const size_t rows = (size_t)B * (size_t)T;
    return kHeaderBytes + align256(rows * kPartialsPerToken * sizeof(float)) + align256(rows * sizeof(int32_t));
}

extern "C" int ppo_workspace_init(void *workspace, size_t bytes, void *stream)
{
    if (!workspace) return PPO_ERR_NULL;
    if (bytes < kHeaderBytes) return PPO_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return PPO_ERR_ALIGN;
    PPO_RETURN_IF_CUDA(cudaMemsetAsync(workspace, 0, kHeaderBytes, reinterpret_cast<cudaStream_t>(stream)));
    return PPO_OK;
}

extern "C" int ppo_last_device_status(void *workspace, void *stream, int *status)
{
    if (!workspace || !status) return PPO_ERR_NULL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    PPO_RETURN_IF_CUDA(cudaMemcpyAsync(status, &ws_header(workspace)->status, sizeof(int), cudaMemcpyDeviceToHost, s));
    PPO_RETURN_IF_CUDA(cudaMemsetAsync(&ws_header(workspace)->status, 0, sizeof(int), s));
    PPO_RETURN_IF_CUDA(cudaStreamSynchronize(s));
    return PPO_OK;
}

extern "C" int ppo_truncate_and_score(const int32_t *responses, int32_t B, int32_t T, int32_t eos_id,
                                      int32_t pad_id, const float *scores, float no_eos_score,
                                      int32_t *responses_out, int32_t *eos_index, int32_t *seq_len,
                                      uint8_t *mask, float *scores_out, void *stream)
{
    if (B < 0 || T <= 0) return PPO_ERR_SHAPE;
    if (eos_id == pad_id) return PPO_ERR_PARAM;
    if (B == 0) return PPO_OK;
    if (!responses || (scores_out && !scores)) return PPO_ERR_NULL;
    const int warps_per_block = 4;
    const unsigned grid = (unsigned)((B + warps_per_block - 1) / warps_per_block);
    truncate_kernel<<<grid, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        responses, B, T, eos_id, pad_id, scores, no_eos_score, responses_out, eos_index, seq_len, mask, scores_out);
    return launch_status();
}

extern "C" int ppo_kl_rewards(const float *logprob, const float *ref_logprob, const uint8_t *mask,
                              const int32_t *seq_len, const float *scores, int32_t B, int32_t T,
                              float kl_coef, float *kl, float *rewards, void *stream)
{
    if (B < 0 || T <= 0) return PPO_ERR_SHAPE;
    if (!finite_f(kl_coef)) return PPO_ERR_PARAM;
    if (B == 0) return PPO_OK;
    if (!logprob || !ref_logprob || !mask || (!kl && !rewards) || (rewards && (!seq_len || !scores)))
        return PPO_ERR_NULL;
    const int64_t n = (int64_t)B * T;
    kl_rewards_kernel<<<(unsigned)((n + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        logprob, ref_logprob, mask, seq_len, scores, B, T, kl_coef, kl, rewards);
    return launch_status();
}

extern "C" int ppo_gae(const float *rewards, const float *values, const int32_t *seq_len, int32_t B, int32_t T,
                       float gamma, float lam, float *advantages, float *returns, void *stream)
{
    if (B < 0 || T <= 0) return PPO_ERR_SHAPE;
    if (!finite_f(gamma) || !finite_f(lam)) return PPO_ERR_PARAM;
    if (B == 0) return PPO_OK;
    if (!rewards || !values || !seq_len || !advantages || !returns) return PPO_ERR_NULL;
    const unsigned grid = (unsigned)((B + 3) / 4);
    gae_kernel<<<grid, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        rewards, values, seq_len, B, T, (double)gamma, (double)gamma * (double)lam, advantages, returns);
    return launch_status();
}

extern "C" int ppo_whiten(const float *x, const uint8_t *mask, int64_t n_elems, int shift_mean, float eps,
                          float *out, float *stats3, void *workspace, void *stream)
{
    if (n_elems < 0) return PPO_ERR_SHAPE;
    if (!(eps >= 0.f) || !finite_f(eps)) return PPO_ERR_PARAM;
    if (n_elems == 0) return PPO_OK;
    if (!x || !out) return PPO_ERR_NULL;
    int *status = workspace ? &ws_header(workspace)->status : nullptr;
    whiten_kernel<<<1, kWhitenThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(x, mask, n_elems, shift_mean, eps,
                                                                                    out, stats3, status);
    return launch_status();
}

extern "C" int ppo_loss_from_logprob(const float *new_logprob, const float *entropy, int32_t B, int32_t T,
                                     const uint8_t *mask, const float *old_logprob, const float *advantages,
                                     const float *values_new, const float *values_old, const float *returns,
                                     const ppo_params *p, float *losses, float *dlogprob, float *dvalues,
                                     void *workspace, void *stream)
{
    if (B <= 0 || T <= 0 || (int64_t)B * T >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    if (!new_logprob || !mask || !old_logprob || !advantages || !values_new || !values_old || !returns || !p ||
        !losses || !dvalues || !workspace)
        return PPO_ERR_NULL;
    if (!(p->cliprange >= 0.f) || !(p->cliprange_value >= 0.f) || !finite_f(p->vf_coef)) return PPO_ERR_PARAM;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return PPO_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int64_t rows = (int64_t)B * T;
    int rc = launch_loss_prepare(mask, rows, workspace, s);
    if (rc) return rc;
    loss_from_logprob_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(
        new_logprob, entropy, rows, mask, old_logprob, advantages, values_new, values_old, returns, p->cliprange,
        p->cliprange_value, p->vf_coef, ws_header(workspace), ws_partials(workspace), dlogprob, dvalues);
    rc = launch_status();
    if (rc) return rc;
    return launch_loss_finalize(rows, p->vf_coef, losses, workspace, s);
}

// ---------------------------------------------------------------- allocation-free variant
// Scratch for ppo_loss_from_logprob_static lives in this file-scope device array instead of a
// caller-provided workspace: same layout as a workspace (header, per-token partials, row order).
// Every GPU that loads the library carries these bytes until the process exits.
namespace {
constexpr size_t kStaticPartialBytes = ((size_t)PPO_STATIC_MAX_TOKENS * kPartialsPerToken * sizeof(float) + 255) & ~size_t(255);
constexpr size_t kStaticOrderBytes = ((size_t)PPO_STATIC_MAX_TOKENS * sizeof(int32_t) + 255) & ~size_t(255);
constexpr size_t kStaticScratchBytes = kHeaderBytes + kStaticPartialBytes + kStaticOrderBytes;
}   // namespace

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on the current device. In host code the array's name is only a
// handle for the runtime, not an address a kernel could use; cudaGetSymbolAddress translates it,
// once per device, with that device current.
static int static_scratch_address(void **out)
{
    static void *cached[64] = {nullptr};
    int dev = 0;
    PPO_RETURN_IF_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PPO_ERR_UNSUPPORTED;
    if (!cached[dev]) {
        void *p = nullptr;
        PPO_RETURN_IF_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        cached[dev] = p;
    }
    *out = cached[dev];
    return PPO_OK;
}

extern "C" int ppo_loss_from_logprob_static(const float *new_logprob, const float *entropy, int32_t B, int32_t T,
                                            const uint8_t *mask, const float *old_logprob, const float *advantages,
                                            const float *values_new, const float *values_old, const float *returns,
                                            const ppo_params *p, float *losses, float *dlogprob, float *dvalues,
                                            void *stream)
{
    if (B <= 0 || T <= 0) return PPO_ERR_SHAPE;
    if ((int64_t)B * T > PPO_STATIC_MAX_TOKENS) return PPO_ERR_UNSUPPORTED;   // beyond the built-in scratch
    if (!new_logprob || !mask || !old_logprob || !advantages || !values_new || !values_old || !returns || !p ||
        !losses || !dvalues)
        return PPO_ERR_NULL;
    if (!(p->cliprange >= 0.f) || !(p->cliprange_value >= 0.f) || !finite_f(p->vf_coef)) return PPO_ERR_PARAM;
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int64_t rows = (int64_t)B * T;
    // the array keeps whatever the previous call left: the prologue rewrites the token count, the work
    // counters and the row order, the token kernel rewrites every partial it later sums; the sticky
    // status word is the one thing that has to be cleared by hand
    PPO_RETURN_IF_CUDA(cudaMemsetAsync(&ws_header(scratch)->status, 0, sizeof(int), s));
    rc = launch_loss_prepare(mask, rows, scratch, s);
    if (rc) return rc;
    loss_from_logprob_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(
        new_logprob, entropy, rows, mask, old_logprob, advantages, values_new, values_old, returns, p->cliprange,
        p->cliprange_value, p->vf_coef, ws_header(scratch), ws_partials(scratch), dlogprob, dvalues);
    rc = launch_status();
    if (rc) return rc;
    return launch_loss_finalize(rows, p->vf_coef, losses, scratch, s);
}
