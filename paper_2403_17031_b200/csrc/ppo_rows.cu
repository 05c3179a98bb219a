// Row kernels: the two steps that stream the [rows, V] logits, and their C entry points.
//   ppo_logprob_entropy  -- one read of every row (single-pass softmax statistics)
//   ppo_loss_fwd_bwd     -- one read and one write of every real row: the row is parked in
//                           shared memory between the statistics pass and the gradient pass
// The entry points prefer the bulk-copy row engine (ppo_rows_bulk.cu). The kernels in this file
// load straight into registers and serve every shape the engine does not take: rows that are not
// 16-byte aligned, V not a multiple of the pack size, rows larger than shared memory, and the
// forward-only loss call. One thread block owns one row at a time; fp32 accumulation in base-2
// units (one ex2 per element); warp-shuffle + shared-memory merge of the per-thread states;
// per-token scalar math in fp64 by one thread.
#include "ppo_rows.cuh"

namespace ppo {

// ---------------------------------------------------------------- step 1 kernel
// One block per row (grid = rows). Kept free of loop-carried state so that it fits 32 registers:
// eight blocks of 256 threads per SM.
template <typename T, bool VECTOR, bool ENTROPY, int THREADS>
__device__ __forceinline__ void logprob_entropy_row(const T *__restrict__ logits, int V, int64_t row_stride,
                                                    const int32_t *__restrict__ tokens,
                                                    const uint8_t *__restrict__ mask, float c,
                                                    float *__restrict__ logprob, float *__restrict__ entropy,
                                                    float *__restrict__ lse, int *status, float *red)
{
    const int64_t row = blockIdx.x;
    if (mask && !mask[row]) {
        if (threadIdx.x == 0) {
            logprob[row] = 0.f;
            if (entropy) entropy[row] = 0.f;
            if (lse) lse[row] = 0.f;
        }
        return;
    }
    const T *src = logits + row * row_stride;
    SoftmaxState st;
    if (VECTOR) {
        const float m_common = row_reference<T>(src, c);
        st = row_statistics<T, true, false, ENTROPY, THREADS, 4>(src, V, c, nullptr, m_common);
        st = block_merge_common<THREADS>(st, m_common, red);
    } else {
        st = row_statistics<T, false, false, ENTROPY, THREADS, 4>(src, V, c, nullptr, 0.f);
        st = block_merge<THREADS>(st, red);
    }
    if (threadIdx.x == 0) {
        const int tok = tokens[row];
        const bool bad = tok < 0 || tok >= V;
        const float xtok = bad ? 0.f : Pack<T>::load1(src + tok);
        const float l2s = log2f(st.s);
        float lp = (fmaf(xtok, c, -st.m) - l2s) * kLn2;
        float H = (l2s - st.u / st.s) * kLn2;
        float L = (st.m + l2s) * kLn2;
        if (bad) {
            lp = H = L = __int_as_float(0x7fc00000);
            if (status) atomicOr(status, PPO_DEV_BAD_TOKEN);
        }
        logprob[row] = lp;
        if (entropy) entropy[row] = H;
        if (lse) lse[row] = L;
    }
}

template <typename T, bool VECTOR, bool ENTROPY, int THREADS>
__global__ void __launch_bounds__(THREADS)
logprob_entropy_kernel(const T *__restrict__ logits, int V, int64_t row_stride, const int32_t *__restrict__ tokens,
                       const uint8_t *__restrict__ mask, float c, float *__restrict__ logprob,
                       float *__restrict__ entropy, float *__restrict__ lse, int *status)
{
    __shared__ float red[96];
    logprob_entropy_row<T, VECTOR, ENTROPY, THREADS>(logits, V, row_stride, tokens, mask, c, logprob, entropy, lse,
                                                     status, red);
}

// Step 1 for the policy and the frozen reference in one launch (grid.y = 2): same tokens, same shape.
// y = 0: policy logits -> log-prob and entropy; y = 1: reference logits -> log-prob only. One launch
// instead of two saves a launch boundary, at which the SMs drain and refill.
// seq_T > 0: the rows are [B, seq_T] responses and everything after a sequence's first EOS is padding (the EOS
// trick of the paper's detail "EOS trick"; the token-level kernel that follows writes the same mask): such a
// row's logits are not read and its outputs are 0, as with mask[row] == 0.
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS)
logprob_pair_kernel(const T *__restrict__ policy_logits, const T *__restrict__ ref_logits, int V,
                    const int32_t *__restrict__ tokens, const uint8_t *__restrict__ mask, int seq_T, int eos_id,
                    float c, float *__restrict__ logprob, float *__restrict__ entropy,
                    float *__restrict__ ref_logprob, int *status, int *flags2)
{
    __shared__ float red[96];
    // ppo_step: the hand-over flags between the two kernels that follow start at 0. The token-level kernel may be
    // scheduled as soon as every block of this grid has passed the trigger below, and part of it runs before it
    // waits for this grid's end, so the block that clears the flags makes the stores visible before its trigger.
    if (flags2 && blockIdx.x == 0 && blockIdx.y == 0) {
        if (threadIdx.x == 0) {
            flags2[0] = 0;
            flags2[1] = 0;
            __threadfence();
        }
        __syncthreads();
    }
    grid_dependents_may_launch();   // the token-level kernel may be scheduled as this grid drains
    if (seq_T > 0) {
        const int64_t row = blockIdx.x;
        const int t = (int)(row % seq_T);
        const int32_t *r = tokens + (row - t);
        int hit = 0;
        for (int i = threadIdx.x; i < t; i += THREADS) hit |= r[i] == eos_id;
        if (__syncthreads_or(hit)) {
            if (threadIdx.x == 0) {
                if (blockIdx.y == 0) {
                    logprob[row] = 0.f;
                    entropy[row] = 0.f;
                } else {
                    ref_logprob[row] = 0.f;
                }
            }
            return;
        }
    }
    if (blockIdx.y == 0)
        logprob_entropy_row<T, true, true, THREADS>(policy_logits, V, V, tokens, mask, c, logprob, entropy, nullptr,
                                                    status, red);
    else
        logprob_entropy_row<T, true, false, THREADS>(ref_logits, V, V, tokens, mask, c, ref_logprob, nullptr,
                                                     nullptr, status, red);
}

// ---------------------------------------------------------------- step 6 kernel

template <typename T, bool VECTOR, int THREADS>
__device__ __forceinline__ void fill_row_zero(T *dst, int V)
{
    if (VECTOR) {
        uint4 *d4 = reinterpret_cast<uint4 *>(dst);
        const int nvec = V / Pack<T>::N;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
        for (int i = threadIdx.x; i < nvec; i += THREADS) st_stream(d4 + i, z);
    } else {
        for (int j = threadIdx.x; j < V; j += THREADS) Pack<T>::store1(dst + j, 0.f);
    }
}

// ROW_IN_SMEM: pass 2 reads the row back from shared memory (every thread re-reads exactly the
// packs it parked itself); otherwise it re-reads global memory (served by L2 when the row is
// still resident there).
template <typename T, bool VECTOR, bool ROW_IN_SMEM, int THREADS>
__global__ void __launch_bounds__(THREADS)
loss_rows_kernel(const LossArgs a)
{
    extern __shared__ uint4 row_stage[];
    __shared__ float red[96];
    __shared__ float bc[2];
    const T *logits = reinterpret_cast<const T *>(a.logits);
    T *dlogits = reinterpret_cast<T *>(a.dlogits);
    const int V = a.V;
    const double n = (double)(*a.n_tokens);

    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x) {
        T *dst = dlogits ? dlogits + row * (int64_t)V : nullptr;
        float *part = a.partials + row * kPartialsPerToken;
        if (!a.mask[row]) {
            if (dst) fill_row_zero<T, VECTOR, THREADS>(dst, V);
            if (threadIdx.x == 0) {
                if (a.dvalues) a.dvalues[row] = 0.f;
                if (a.new_logprob) a.new_logprob[row] = 0.f;
                if (a.entropy) a.entropy[row] = 0.f;
                if (a.dlogprob) a.dlogprob[row] = 0.f;
                float4 *p4 = reinterpret_cast<float4 *>(part);
                p4[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                p4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            continue;
        }
        const T *src = logits + row * (int64_t)V;
        const int tok = a.tokens[row];
        const bool bad = tok < 0 || tok >= V;
        float xtok = 0.f, t_old = 0.f, t_adv = 0.f, t_vn = 0.f, t_vo = 0.f, t_ret = 0.f;
        if (threadIdx.x == 0) {   // per-token scalars: fetched now, used after the row reduction
            if (!bad) xtok = Pack<T>::load1(src + tok);
            if (a.g_ext) {
                t_old = a.g_ext[row];
            } else {
                t_old = a.old_logprob[row];
                t_adv = a.advantages[row];
                t_vn = a.values_new[row];
                t_vo = a.values_old[row];
                t_ret = a.returns[row];
            }
        }
        SoftmaxState st;
        if (VECTOR) {
            const float m_common = row_reference<T>(src, a.c);
            st = row_statistics<T, true, ROW_IN_SMEM, true, THREADS, 4>(src, V, a.c, row_stage, m_common);
            st = block_merge_common<THREADS>(st, m_common, red);
        } else {
            st = row_statistics<T, false, ROW_IN_SMEM, true, THREADS, 4>(src, V, a.c, row_stage, 0.f);
            st = block_merge<THREADS>(st, red);
        }
        if (threadIdx.x == 0) {
            const float l2s = log2f(st.s);
            float lp = (fmaf(xtok, a.c, -st.m) - l2s) * kLn2;
            float H = (l2s - st.u / st.s) * kLn2;
            if (bad) {
                lp = H = __int_as_float(0x7fc00000);
                if (a.status) atomicOr(a.status, PPO_DEV_BAD_TOKEN);
            }
            TokenLoss tl;
            if (a.g_ext) {   // the gradient on the log-prob is an input (a bad token still poisons its row)
                tl.g = bad ? lp : t_old;
                tl.dvalue = tl.pg = tl.vf = tl.kl = tl.pg_clipped = tl.vf_clipped = 0.f;
            } else {
                tl = token_loss(lp, t_old, t_adv, t_vn, t_vo, t_ret, a.eps, a.eps_v, a.c1, n);
            }
            if (a.dvalues) a.dvalues[row] = tl.dvalue;
            if (a.new_logprob) a.new_logprob[row] = lp;
            if (a.entropy) a.entropy[row] = H;
            if (a.dlogprob) a.dlogprob[row] = tl.g;
            float4 *p4 = reinterpret_cast<float4 *>(part);
            p4[0] = make_float4(tl.pg, tl.vf, tl.kl, tl.pg_clipped);
            p4[1] = make_float4(tl.vf_clipped, H, 0.f, 0.f);
            bc[0] = st.m + l2s;          // log2-sum-exp
            bc[1] = tl.g * a.inv_tau;    // gradient scale
        }
        __syncthreads();
        const float Y = bc[0], gs = bc[1];
        if (dst) {
            if (gs == 0.f) {
                fill_row_zero<T, VECTOR, THREADS>(dst, V);
            } else {
                // -gs * 2^(y - Y) = -+ 2^(y - Y + log2|gs|): the scale rides in the exponent
                const float off = log2f(fabsf(gs)) - Y;
                const bool neg = gs > 0.f;
                if (VECTOR) {
                    constexpr int N = Pack<T>::N;
                    const uint4 *src4 = ROW_IN_SMEM ? row_stage : reinterpret_cast<const uint4 *>(src);
                    uint4 *dst4 = reinterpret_cast<uint4 *>(dst);
                    const int nvec = V / N;
                    if (neg) {
#pragma unroll 2
                        for (int i = threadIdx.x; i < nvec; i += THREADS) {
                            float x[N], d[N];
                            Pack<T>::unpack_raw(src4[i], x);
#pragma unroll
                            for (int k = 0; k < N; ++k) d[k] = -ex2(fmaf(x[k], a.c, off));
                            st_stream(dst4 + i, Pack<T>::pack(d));
                        }
                    } else {
#pragma unroll 2
                        for (int i = threadIdx.x; i < nvec; i += THREADS) {
                            float x[N], d[N];
                            Pack<T>::unpack_raw(src4[i], x);
#pragma unroll
                            for (int k = 0; k < N; ++k) d[k] = ex2(fmaf(x[k], a.c, off));
                            st_stream(dst4 + i, Pack<T>::pack(d));
                        }
                    }
                    // the thread that wrote the pack holding the sampled token adds the one-hot term
                    if (!bad && threadIdx.x == (tok / N) % THREADS) {
                        const float e = ex2(fmaf(Pack<T>::load1(src + tok), a.c, off));
                        Pack<T>::store1(dst + tok, gs + (neg ? -e : e));
                    }
                } else {
                    const T *src1 = ROW_IN_SMEM ? reinterpret_cast<const T *>(row_stage) : src;
                    for (int j = threadIdx.x; j < V; j += THREADS) {
                        const float e = ex2(fmaf(Pack<T>::load1(src1 + j), a.c, off));
                        float d = neg ? -e : e;
                        if (j == tok) d += gs;
                        Pack<T>::store1(dst + j, d);
                    }
                }
            }
        }
        __syncthreads();   // bc and the staged row are reused by the next row
    }
}

// ---------------------------------------------------------------- host side

template <typename T>
static int launch_logprob(const void *logits, int64_t rows, int V, int64_t row_stride, const int32_t *tokens,
                          const uint8_t *mask, float c, float *logprob, float *entropy, float *lse, int *status,
                          cudaStream_t s)
{
    constexpr int THREADS = 256;
    const bool vec = aligned16(logits) && (row_stride * sizeof(T)) % 16 == 0 && V % Pack<T>::N == 0;
    const unsigned grid = (unsigned)rows;   // rows < 2^31 is checked by the caller
    const T *lg = reinterpret_cast<const T *>(logits);
#define PPO_LAUNCH_LP(VEC, ENT)                                                                       \
    logprob_entropy_kernel<T, VEC, ENT, THREADS><<<grid, THREADS, 0, s>>>(lg, V, row_stride, tokens, mask, c, \
                                                                          logprob, entropy, lse, status)
    if (vec) {
        if (entropy) PPO_LAUNCH_LP(true, true); else PPO_LAUNCH_LP(true, false);
    } else {
        if (entropy) PPO_LAUNCH_LP(false, true); else PPO_LAUNCH_LP(false, false);
    }
#undef PPO_LAUNCH_LP
    return launch_status();
}

// PPO_ERR_UNSUPPORTED when the pointers or the shape do not allow 16-byte packs (the caller then makes two calls)
int launch_logprob_pair(const void *policy_logits, const void *ref_logits, int dtype, int64_t rows, int V,
                        const int32_t *tokens, const uint8_t *mask, int seq_T, int eos_id, float c, float *logprob,
                        float *entropy, float *ref_logprob, WorkspaceHeader *hdr, bool clear_flags, cudaStream_t s)
{
    int *status = hdr ? &hdr->status : nullptr, *flags2 = (hdr && clear_flags) ? &hdr->order_ready : nullptr;
    static_assert(offsetof(WorkspaceHeader, adv_ready) == offsetof(WorkspaceHeader, order_ready) + sizeof(int),
                  "the two flags are cleared as a pair");
    constexpr int THREADS = 256;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    const int N = dtype == PPO_F32 ? 4 : 8;
    if (!aligned16(policy_logits) || !aligned16(ref_logits) || ((size_t)V * es) % 16 != 0 || V % N != 0)
        return PPO_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)rows, 2);
    if (dtype == PPO_F32)
        logprob_pair_kernel<float, THREADS><<<grid, THREADS, 0, s>>>(
            reinterpret_cast<const float *>(policy_logits), reinterpret_cast<const float *>(ref_logits), V, tokens, mask,
            seq_T, eos_id, c, logprob, entropy, ref_logprob, status, flags2);
    else
        logprob_pair_kernel<__nv_bfloat16, THREADS><<<grid, THREADS, 0, s>>>(
            reinterpret_cast<const __nv_bfloat16 *>(policy_logits), reinterpret_cast<const __nv_bfloat16 *>(ref_logits),
            V, tokens, mask, seq_T, eos_id, c, logprob, entropy, ref_logprob, status, flags2);
    return launch_status();
}

constexpr size_t kMaxDynSmem = 227 * 1024;

template <typename T, bool VECTOR, bool ROW_IN_SMEM, int THREADS>
static int launch_loss_variant(const LossArgs &a, size_t smem, cudaStream_t s)
{
    auto kern = loss_rows_kernel<T, VECTOR, ROW_IN_SMEM, THREADS>;
    if (smem > 48 * 1024)
        PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned grid = (unsigned)(a.rows < (int64_t)1 << 30 ? a.rows : (int64_t)1 << 30);
    kern<<<grid, THREADS, smem, s>>>(a);
    return launch_status();
}

template <typename T>
static int launch_loss(const LossArgs &a, cudaStream_t s)
{
    const bool vec = aligned16(a.logits) && (a.dlogits == nullptr || aligned16(a.dlogits)) &&
                     a.V % Pack<T>::N == 0;
    const size_t row_bytes = (size_t)a.V * sizeof(T);
    // Two blocks per SM when the row is small enough (they overlap each other's load, compute
    // and store phases); one big block per SM while the row still fits; else re-read via L2.
    const int mode = option_value(PPO_OPT_LOSS_ROW_CACHE);
    const bool fits2 = row_bytes <= 112 * 1024, fits1 = row_bytes + 1024 <= kMaxDynSmem;
    bool in_smem = a.dlogits != nullptr && (fits2 || fits1);
    if (mode == 1) in_smem = fits1;
    if (mode == 2) in_smem = false;
    if (in_smem) {
        if (fits2) {
            return vec ? launch_loss_variant<T, true, true, 512>(a, row_bytes, s)
                       : launch_loss_variant<T, false, true, 512>(a, row_bytes, s);
        }
        return vec ? launch_loss_variant<T, true, true, 1024>(a, row_bytes, s)
                   : launch_loss_variant<T, false, true, 1024>(a, row_bytes, s);
    }
    return vec ? launch_loss_variant<T, true, false, 512>(a, 0, s)
               : launch_loss_variant<T, false, false, 512>(a, 0, s);
}

}   // namespace ppo

using namespace ppo;

extern "C" int ppo_logprob_entropy(const void *logits, int dtype, int64_t rows, int64_t V, int64_t row_stride,
                                   const int32_t *tokens, const uint8_t *mask, float temperature,
                                   float *logprob, float *entropy, float *lse, void *workspace, void *stream)
{
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (rows < 0 || rows >= ((int64_t)1 << 31) || V <= 0 || V >= ((int64_t)1 << 31) || row_stride < V)
        return PPO_ERR_SHAPE;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    if (rows == 0) return PPO_OK;
    if (!logits || !tokens || !logprob) return PPO_ERR_NULL;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return PPO_ERR_ALIGN;
    int *status = workspace ? &ws_header(workspace)->status : nullptr;
    const float c = kLog2e / temperature;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (option_value(PPO_OPT_ROW_ENGINE) == 2) {
        const int rc = launch_logprob_bulk(logits, dtype, rows, (int)V, row_stride, tokens, mask, c, logprob, entropy,
                                           lse, status, s);
        if (rc != PPO_ERR_UNSUPPORTED) return rc;
    }
    if (dtype == PPO_F32)
        return launch_logprob<float>(logits, rows, (int)V, row_stride, tokens, mask, c, logprob, entropy, lse,
                                     status, s);
    return launch_logprob<__nv_bfloat16>(logits, rows, (int)V, row_stride, tokens, mask, c, logprob, entropy, lse,
                                         status, s);
}

extern "C" int ppo_loss_fwd_bwd(const void *logits, int dtype, int32_t B, int32_t T, int64_t V,
                                const int32_t *tokens, const uint8_t *mask, const float *old_logprob,
                                const float *advantages, const float *values_new, const float *values_old,
                                const float *returns, const ppo_params *p, float *losses, void *dlogits,
                                float *dvalues, float *new_logprob, float *entropy, float *dlogprob,
                                void *workspace, void *stream)
{
    return loss_fwd_bwd_prepared(logits, dtype, B, T, V, tokens, mask, old_logprob, advantages, values_new, values_old,
                                 returns, p, losses, dlogits, dvalues, new_logprob, entropy, dlogprob, workspace, stream,
                                 false);
}

extern "C" int ppo_loss_fwd_bwd_next_epoch(const void *logits, int dtype, int32_t B, int32_t T, int64_t V,
                                           const int32_t *tokens, const uint8_t *mask, const float *old_logprob,
                                           const float *advantages, const float *values_new,
                                           const float *values_old, const float *returns, const ppo_params *p,
                                           float *losses, void *dlogits, float *dvalues, float *new_logprob,
                                           float *entropy, float *dlogprob, void *workspace, void *stream)
{
    return loss_fwd_bwd_prepared(logits, dtype, B, T, V, tokens, mask, old_logprob, advantages, values_new, values_old,
                                 returns, p, losses, dlogits, dvalues, new_logprob, entropy, dlogprob, workspace, stream,
                                 false, true);
}

int ppo::loss_fwd_bwd_prepared(const void *logits, int dtype, int32_t B, int32_t T, int64_t V, const int32_t *tokens,
                               const uint8_t *mask, const float *old_logprob, const float *advantages,
                               const float *values_new, const float *values_old, const float *returns,
                               const ppo_params *p, float *losses, void *dlogits, float *dvalues, float *new_logprob,
                               float *entropy, float *dlogprob, void *workspace, void *stream, bool prepared,
                               bool reuse)
{
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (B <= 0 || T <= 0 || V <= 0 || V >= ((int64_t)1 << 31) || (int64_t)B * T >= ((int64_t)1 << 31))
        return PPO_ERR_SHAPE;
    if (!logits || !tokens || !mask || !old_logprob || !advantages || !values_new || !values_old || !returns ||
        !p || !losses || !dvalues || !workspace)
        return PPO_ERR_NULL;
    if (!(p->temperature > 0.f) || !finite_f(p->temperature) || !(p->cliprange >= 0.f) ||
        !(p->cliprange_value >= 0.f) || !finite_f(p->vf_coef))
        return PPO_ERR_PARAM;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es || reinterpret_cast<uintptr_t>(dlogits) % es ||
        reinterpret_cast<uintptr_t>(workspace) % 256)
        return PPO_ERR_ALIGN;
    if (dlogits == logits) return PPO_ERR_PARAM;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int64_t rows = (int64_t)B * T;
    // reuse: the row order of the previous loss call on this workspace serves this call too (same mask): the bulk
    // engine starts at once; the kernels that cannot check this run the prologue as usual
    int rc = (prepared || reuse) ? PPO_OK : launch_loss_prepare(mask, rows, workspace, s);
    if (rc) return rc;
    LossArgs a;
    a.logits = logits;
    a.dlogits = dlogits;
    a.rows = rows;
    a.V = (int)V;
    a.tokens = tokens;
    a.mask = mask;
    a.g_ext = nullptr;
    a.old_logprob = old_logprob;
    a.advantages = advantages;
    a.values_new = values_new;
    a.values_old = values_old;
    a.returns = returns;
    a.dvalues = dvalues;
    a.new_logprob = new_logprob;
    a.entropy = entropy;
    a.dlogprob = dlogprob;
    a.partials = ws_partials(workspace);
    a.n_tokens = &ws_header(workspace)->n_tokens;
    a.status = &ws_header(workspace)->status;
    a.c = kLog2e / p->temperature;
    a.inv_tau = 1.0f / p->temperature;
    a.eps = p->cliprange;
    a.eps_v = p->cliprange_value;
    a.c1 = p->vf_coef;
    rc = PPO_ERR_UNSUPPORTED;
    if (option_value(PPO_OPT_ROW_ENGINE) != 1) {
        rc = launch_loss_bulk(a, dtype, workspace, losses, p->vf_coef, !reuse, s, reuse, !prepared);
        if (rc != PPO_ERR_UNSUPPORTED) return rc;      // the engine reduces the partials itself
    }
    if (reuse) {
        rc = launch_loss_prepare(mask, rows, workspace, s);
        if (rc) return rc;
    }
    rc = dtype == PPO_F32 ? launch_loss<float>(a, s) : launch_loss<__nv_bfloat16>(a, s);
    if (rc) return rc;
    return launch_loss_finalize(rows, p->vf_coef, losses, workspace, s);
}

extern "C" int ppo_logprob_bwd(const void *logits, int dtype, int64_t rows, int64_t V, const int32_t *tokens,
                               const uint8_t *mask, const float *dlogprob, float temperature, void *dlogits,
                               float *new_logprob, float *entropy, void *workspace, void *stream)
{
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (rows <= 0 || V <= 0 || V >= ((int64_t)1 << 31) || rows >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    if (!logits || !tokens || !mask || !dlogprob || !dlogits || !workspace) return PPO_ERR_NULL;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es || reinterpret_cast<uintptr_t>(dlogits) % es ||
        reinterpret_cast<uintptr_t>(workspace) % 256)
        return PPO_ERR_ALIGN;
    if (dlogits == logits) return PPO_ERR_PARAM;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int rc = launch_loss_prepare(mask, rows, workspace, s);
    if (rc) return rc;
    LossArgs a = {};
    a.logits = logits;
    a.dlogits = dlogits;
    a.rows = rows;
    a.V = (int)V;
    a.tokens = tokens;
    a.mask = mask;
    a.g_ext = dlogprob;
    a.new_logprob = new_logprob;
    a.entropy = entropy;
    a.partials = ws_partials(workspace);
    a.n_tokens = &ws_header(workspace)->n_tokens;
    a.status = &ws_header(workspace)->status;
    a.c = kLog2e / temperature;
    a.inv_tau = 1.0f / temperature;
    // the kernels end with the reduction of the (all-zero) loss partials; it lands in the header's spare words
    float *sink = reinterpret_cast<float *>(ws_header(workspace)->reserved);
    rc = PPO_ERR_UNSUPPORTED;
    if (option_value(PPO_OPT_ROW_ENGINE) != 1) {
        rc = launch_loss_bulk(a, dtype, workspace, sink, 0.f, true, s);
        if (rc != PPO_ERR_UNSUPPORTED) return rc;
    }
    rc = dtype == PPO_F32 ? launch_loss<float>(a, s) : launch_loss<__nv_bfloat16>(a, s);
    if (rc) return rc;
    return launch_loss_finalize(rows, 0.f, sink, workspace, s);
}

extern "C" int ppo_logprob_entropy_pair(const void *policy_logits, const void *ref_logits, int dtype, int64_t rows,
                                        int64_t V, const int32_t *tokens, const uint8_t *mask, float temperature,
                                        float *logprob, float *entropy, float *ref_logprob, void *workspace,
                                        void *stream)
{
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (rows < 0 || rows >= ((int64_t)1 << 31) || V <= 0 || V >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    if (rows == 0) return PPO_OK;
    if (!policy_logits || !ref_logits || !tokens || !logprob || !ref_logprob) return PPO_ERR_NULL;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(policy_logits) % es || reinterpret_cast<uintptr_t>(ref_logits) % es)
        return PPO_ERR_ALIGN;
    int rc = launch_logprob_pair(policy_logits, ref_logits, dtype, rows, (int)V, tokens, mask, 0, 0, kLog2e / temperature,
                                 logprob, entropy, ref_logprob, workspace ? ws_header(workspace) : nullptr, false,
                                 reinterpret_cast<cudaStream_t>(stream));
    if (rc != PPO_ERR_UNSUPPORTED) return rc;
    // no 16-byte packs in this layout: one launch per tensor
    rc = ppo_logprob_entropy(policy_logits, dtype, rows, V, V, tokens, mask, temperature, logprob, entropy, nullptr,
                             workspace, stream);
    if (rc) return rc;
    return ppo_logprob_entropy(ref_logits, dtype, rows, V, V, tokens, mask, temperature, ref_logprob, nullptr, nullptr,
                               workspace, stream);
}
