// Shared device/host helpers of the PPO hot-path kernels (sm_100a).
#pragma once

#include <cstddef>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "ppo_b200.h"

namespace ppo {

// ---------------------------------------------------------------- workspace layout
// [0, 256)                      WorkspaceHeader
// [256, +align256(rows*8*4))    per-token loss partials, 8 floats per token
// [.., +align256(rows*4))       row order of the loss call: real rows first (ascending), then
//                               masked rows from the back
struct WorkspaceHeader {
    int status;        // PPO_DEV_* bits, sticky until read
    int n_tokens;      // number of mask==1 tokens of the loss call in flight
    int masked_next;   // work counter of the zero-fill phase (reset by every loss call)
    int done_blocks;   // blocks of the loss kernel that have retired (reset by every loss call)
    int step_blocks;   // blocks of ppo_step's token-level kernel that have finished (resets itself)
    int real_next;     // work counter of the loss kernel's mask==1 rows (reset by every loss call)
    int order_ready;   // n_tokens + 1 once token count, counters and row order of the loss call in flight are written
    int adv_ready;     // 1 once the advantages / returns that the loss call reads are written
    int step_blocks2;  // second ticket of ppo_step's token-level kernel (resets itself)
    int masked_tail;   // work counter of the masked rows kept back for blocks that run out of real rows (reset by every loss call)
    int reserved[8];
    // what the row order in this workspace was built from: mask pointer, number of rows, order pointer. A loss call
    // that reuses the order (ppo_loss_fwd_bwd_next_epoch) checks its own arguments against these.
    unsigned long long order_sig[3];
    int reserved2[40];
};
static_assert(offsetof(WorkspaceHeader, order_sig) % 8 == 0, "aligned 64-bit words");
static_assert(sizeof(WorkspaceHeader) == 256, "header is one 256-byte block");

constexpr int kPartialsPerToken = 8;   // pg, vf, kl, pg_clipped, vf_clipped, entropy, unused, unused
constexpr size_t kHeaderBytes = 256;

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

__host__ __device__ inline WorkspaceHeader *ws_header(void *ws) { return reinterpret_cast<WorkspaceHeader *>(ws); }
__host__ __device__ inline float *ws_partials(void *ws)
{
    return reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(ws) + kHeaderBytes);
}
inline int32_t *ws_order(void *ws, int64_t rows)
{
    return reinterpret_cast<int32_t *>(reinterpret_cast<unsigned char *>(ws) + kHeaderBytes +
                                       align256((size_t)rows * kPartialsPerToken * sizeof(float)));
}

inline bool finite_f(float x) { return isfinite(x); }

#define PPO_RETURN_IF_CUDA(expr)                      \
    do {                                              \
        cudaError_t e__ = (expr);                     \
        if (e__ != cudaSuccess) return (int)e__;      \
    } while (0)

inline int launch_status()
{
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PPO_OK : (int)e;
}

// ---------------------------------------------------------------- small device helpers
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegBig = -1.0e30f;   // stands in for -inf: exp2 of it is 0 and 0 * it is 0

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Running softmax statistics of a set of scaled logits y (base-2 units, y = logit*log2(e)/tau):
//   m = reference (>= every y seen),  s = sum 2^(y-m),  u = sum 2^(y-m) * (y-m).
// log2-sum-exp = m + log2 s;  entropy = ln2 * (log2 s - u/s).
struct SoftmaxState {
    float m, s, u;
    __device__ __forceinline__ void init() { m = kNegBig; s = 0.f; u = 0.f; }
    // move the reference up to nm >= m
    __device__ __forceinline__ void rebase(float nm)
    {
        float d = m - nm;
        float a = ex2(d);
        u = a * fmaf(d, s, u);
        s *= a;
        m = nm;
    }
    __device__ __forceinline__ void add(float t /* = y - m, <= ~0 */)
    {
        float e = ex2(t);
        s += e;
        u = fmaf(e, t, u);
    }
};

__device__ __forceinline__ SoftmaxState merge(const SoftmaxState &a, const SoftmaxState &b)
{
    SoftmaxState r;
    r.m = fmaxf(a.m, b.m);
    float da = a.m - r.m, db = b.m - r.m;
    float ea = ex2(da), eb = ex2(db);
    r.s = fmaf(a.s, ea, b.s * eb);
    r.u = fmaf(ea, fmaf(da, a.s, a.u), eb * fmaf(db, b.s, b.u));
    return r;
}

__device__ __forceinline__ SoftmaxState warp_merge(SoftmaxState st)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        SoftmaxState o;
        o.m = __shfl_xor_sync(0xffffffffu, st.m, off);
        o.s = __shfl_xor_sync(0xffffffffu, st.s, off);
        o.u = __shfl_xor_sync(0xffffffffu, st.u, off);
        st = merge(st, o);
    }
    return st;
}

// Block-wide merge; `red` holds 3*32 floats. Result is returned to every thread.
template <int THREADS>
__device__ __forceinline__ SoftmaxState block_merge(SoftmaxState st, float *red)
{
    constexpr int WARPS = THREADS / 32;
    st = warp_merge(st);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (WARPS > 1) {
        if (lane == 0) {
            red[warp] = st.m;
            red[32 + warp] = st.s;
            red[64 + warp] = st.u;
        }
        __syncthreads();
        SoftmaxState t;
        if (lane < WARPS) {
            t.m = red[lane];
            t.s = red[32 + lane];
            t.u = red[64 + lane];
        } else {
            t.init();
        }
        st = warp_merge(t);
        __syncthreads();   // red may be reused by the caller's next row
    }
    return st;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// Block-wide merge for the common case in which every thread kept the same reference m_common:
// then merging is adding s and u. One barrier, which also ORs a "my reference differs" flag over
// the block; if any thread moved its reference (overflow rescue) the general merge runs instead.
// The result is valid in thread 0 only. `red` holds 96 floats and is free again after the
// caller's next block-wide barrier.
template <int THREADS>
__device__ __forceinline__ SoftmaxState block_merge_common(SoftmaxState st, float m_common, float *red)
{
    constexpr int WARPS = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (st.s == 0.f) st.m = m_common;                    // a thread without elements
    const int differs = st.m != m_common;
    const float s = warp_sum_f(st.s), u = warp_sum_f(st.u);
    if (lane == 0) {
        red[warp] = s;
        red[32 + warp] = u;
    }
    if (__syncthreads_or(differs)) {
        __syncthreads();                                 // everyone has left the fast path's use of red
        return block_merge<THREADS>(st, red);
    }
    SoftmaxState r;
    r.m = m_common;
    r.s = 0.f;
    r.u = 0.f;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
            r.s += red[w];
            r.u += red[32 + w];
        }
    }
    return r;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// Block-wide fp64 sum in a fixed order; `red` holds 32 doubles. Result to every thread.
template <int THREADS>
__device__ __forceinline__ double block_sum(double v, double *red)
{
    constexpr int WARPS = THREADS / 32;
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = (lane < WARPS) ? red[lane] : 0.0;
    t = warp_sum(t);
    __syncthreads();
    return t;
}

// ---------------------------------------------------------------- per-token PPO loss terms
struct TokenLoss {
    float g;        // d loss / d new_logprob
    float dvalue;   // d loss / d value
    float pg, vf, kl, pg_clipped, vf_clipped;
};

// Clipped surrogate of one real token (Table "PPO hyperparameters": epsilon). fp32: the ratio is one
// ex2, so that this sits cheaply on the critical path between the two passes over a row; inv_n = 1/n.
struct PolicyTerm {
    float g;        // d loss / d new_logprob
    float pg, kl, pg_clipped;
};

__device__ __forceinline__ PolicyTerm policy_term(float lp_new, float lp_old, float adv, float eps, float inv_n)
{
    PolicyTerm o;
    const float lr = lp_new - lp_old;
    const float rho = ex2(lr * kLog2e);
    const float lo = 1.f - eps, hi = 1.f + eps;
    const float rc = rho < lo ? lo : (rho > hi ? hi : rho);
    const float l1 = -adv * rho, l2 = -adv * rc;
    const bool pclip = l2 > l1;
    o.pg = pclip ? l2 : l1;
    o.g = pclip ? 0.f : l1 * inv_n;
    o.pg_clipped = pclip ? 1.f : 0.f;
    o.kl = 0.5f * lr * lr;
    return o;
}

// Clipped value loss of one real token (epsilon-hat, c1, value-loss clipping on). Evaluated in fp64
// from the fp32 inputs so that the branch decision does not depend on fp32 rounding.
struct ValueTerm {
    float dvalue;   // d loss / d value
    float vf, vf_clipped;
};

__device__ __forceinline__ ValueTerm value_term(float v, float v_old, float ret, float eps_v, float c1, double inv_n)
{
    ValueTerm o;
    const double dv = v, dvo = v_old, dr = ret;
    const double vlo = dvo - (double)eps_v, vhi = dvo + (double)eps_v;
    const double vc = dv < vlo ? vlo : (dv > vhi ? vhi : dv);
    const double e1 = (dv - dr) * (dv - dr), e2 = (vc - dr) * (vc - dr);
    const bool vclip = e2 > e1;
    o.vf = (float)(vclip ? e2 : e1);
    o.vf_clipped = vclip ? 1.f : 0.f;
    o.dvalue = vclip ? 0.f : (float)((double)c1 * (dv - dr) * inv_n);
    return o;
}

__device__ __forceinline__ TokenLoss token_loss(float lp_new, float lp_old, float adv, float v, float v_old,
                                               float ret, float eps, float eps_v, float c1, double n)
{
    const double inv_n = 1.0 / n;
    const PolicyTerm pt = policy_term(lp_new, lp_old, adv, eps, (float)inv_n);
    const ValueTerm vt = value_term(v, v_old, ret, eps_v, c1, inv_n);
    TokenLoss o;
    o.g = pt.g;
    o.pg = pt.pg;
    o.kl = pt.kl;
    o.pg_clipped = pt.pg_clipped;
    o.dvalue = vt.dvalue;
    o.vf = vt.vf;
    o.vf_clipped = vt.vf_clipped;
    return o;
}

// Sum the per-token partials in a fixed order (thread t takes rows t, t+NT, ...; fp64) and write the
// eight loss scalars. Called by all NT threads of one block; `red` holds 6*32 doubles; `sync` is a
// barrier over exactly those NT threads.
template <int NT, typename SyncFn>
__device__ __forceinline__ void reduce_loss_partials(const float *partials, int64_t rows, int n_tokens, float vf_coef,
                                                     float *losses, double *red, int t, SyncFn sync)
{
    double acc[6] = {0, 0, 0, 0, 0, 0};
    // the loads of four rows are issued before the first sum needs one (the block that runs this is
    // the only one left: nothing else hides the latency); the order of the additions stays r = t, t + NT, ...
    constexpr int kBatch = 4;
    for (int64_t r = t; r < rows; r += kBatch * (int64_t)NT) {
        float4 p0[kBatch], p1[kBatch];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const int64_t rq = r + q * (int64_t)NT;
            p0[q] = p1[q] = make_float4(0.f, 0.f, 0.f, 0.f);   // past the end: adds +0, which changes no sum
            if (rq < rows) {
                const float4 *src = reinterpret_cast<const float4 *>(partials + rq * kPartialsPerToken);
                p0[q] = __ldcg(src);
                p1[q] = __ldcg(src + 1);
            }
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            acc[0] += p0[q].x; acc[1] += p0[q].y; acc[2] += p0[q].z; acc[3] += p0[q].w;
            acc[4] += p1[q].x; acc[5] += p1[q].y;
        }
    }
    const int lane = t & 31, warp = t >> 5;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        acc[k] = warp_sum(acc[k]);
        if (lane == 0) red[k * 32 + warp] = acc[k];
    }
    sync();
    if (warp == 0) {
        double tot[6];
#pragma unroll
        for (int k = 0; k < 6; ++k) tot[k] = warp_sum(lane < NT / 32 ? red[k * 32 + lane] : 0.0);
        if (lane == 0) {
            const double n = (double)n_tokens;
            const double inv = n > 0.0 ? 1.0 / n : 0.0;
            const double pg = tot[0] * inv, vf = 0.5 * tot[1] * inv;
            losses[PPO_LOSS_PG] = (float)pg;
            losses[PPO_LOSS_VF] = (float)vf;
            losses[PPO_LOSS_TOTAL] = (float)(pg + (double)vf_coef * vf);
            losses[PPO_LOSS_APPROX_KL] = (float)(tot[2] * inv);
            losses[PPO_LOSS_PG_CLIPFRAC] = (float)(tot[3] * inv);
            losses[PPO_LOSS_VF_CLIPFRAC] = (float)(tot[4] * inv);
            losses[PPO_LOSS_ENTROPY] = (float)(tot[5] * inv);
            losses[PPO_LOSS_N] = (float)n;
        }
    }
}

// Hand-over of results between two kernels that overlap in time (the loss kernel of ppo_step is launched
// while the token-level kernel before it is still running, see launch_dependent): the writer publishes
// with flag_set after its data, the reader polls with flag_wait before it touches them. The wait is
// bounded (~1 s); when it runs out the status word gets PPO_DEV_TIMEOUT and the caller carries on.
// PPO_TEST_WITHHOLD_FLAGS (never defined in the product build): a test build in which the flags whose bit is set
// (1 = order_ready, 2 = adv_ready) are never published, so that the bounded waits of the reader run out.
#ifndef PPO_TEST_WITHHOLD_FLAGS
#define PPO_TEST_WITHHOLD_FLAGS 0
#endif
enum FlagKind { kFlagOrder = 1, kFlagAdv = 2 };

__device__ __forceinline__ void flag_set(int *flag, int value /* non-zero */, FlagKind kind)
{
    if (PPO_TEST_WITHHOLD_FLAGS & kind) return;
    __threadfence();
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(value) : "memory");
}

#ifndef PPO_WAIT_TRIES
constexpr uint32_t kFlagWaitTries = 1u << 20;
#else
constexpr uint32_t kFlagWaitTries = PPO_WAIT_TRIES;   // a test build makes the waits short
#endif
// returns the flag's (non-zero) value, or 0 after the wait ran out
__device__ __forceinline__ int flag_wait(const int *flag, int *status)
{
    for (uint32_t it = 0; it < kFlagWaitTries; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v) return v;
        __nanosleep(200);
    }
    if (status) atomicOr(status, PPO_DEV_TIMEOUT);
    return 0;
}

// Programmatic dependent launch: a kernel launched with launch_dependent() may be scheduled while the
// kernel before it in the stream is still running, but only once every block of that kernel has executed
// grid_dependents_may_launch() or has exited - so the earlier kernel is resident and will finish, and the
// later one may wait (flag_wait) for what it produces. The instruction does nothing when no dependent
// launch follows.
__device__ __forceinline__ void grid_dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;"); }
// in a kernel launched with launch_dependent(): returns once the kernel before it has completed and its
// writes are visible (returns at once in a kernel launched the ordinary way)
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
    if (e != cudaSuccess) {   // attribute not accepted in this context: ordinary launch (same results, no overlap)
        (void)cudaGetLastError();
        cfg.numAttrs = 0;
        e = cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
    }
    return e;
}

// launchers shared between translation units
// all token-level steps of ppo_step in one launch (EOS trick, KL rewards, GAE, loss prologue, whitening)
// ppo_loss_fwd_bwd without its prologue launch (the caller has already run the prologue on this mask)
int loss_fwd_bwd_prepared(const void *logits, int dtype, int32_t B, int32_t T, int64_t V, const int32_t *tokens,
                          const uint8_t *mask, const float *old_logprob, const float *advantages,
                          const float *values_new, const float *values_old, const float *returns, const ppo_params *p,
                          float *losses, void *dlogits, float *dvalues, float *new_logprob, float *entropy,
                          float *dlogprob, void *workspace, void *stream, bool prepared, bool reuse = false);
int launch_loss_prepare(const uint8_t *mask, int64_t rows, void *workspace, cudaStream_t s);
// the same prologue with the order array at a place of the caller's choice: hdr->n_tokens = number of rows with
// mask 1, order[0 .. n_tokens) = those rows (ascending), order[n_tokens .. rows) = the other rows
int launch_row_order(const uint8_t *mask, int64_t rows, WorkspaceHeader *hdr, int32_t *order, cudaStream_t s);
// step 1 for policy and reference logits in one launch; PPO_ERR_UNSUPPORTED if the layout rules it out
// (also clears the two hand-over flags of the header for the kernels that follow in ppo_step).
// seq_T > 0: rows = B * seq_T responses, and rows after a sequence's first eos_id are padding (skipped, outputs 0)
int launch_logprob_pair(const void *policy_logits, const void *ref_logits, int dtype, int64_t rows, int V,
                        const int32_t *tokens, const uint8_t *mask, int seq_T, int eos_id, float c, float *logprob,
                        float *entropy, float *ref_logprob, WorkspaceHeader *hdr, bool clear_flags, cudaStream_t s);
// flags_cleared: the launch before this one has cleared the header's hand-over flags already
int launch_rollout(const ppo_step_io *io, int B, int T, const ppo_params *p, bool flags_cleared, cudaStream_t s);
int launch_loss_finalize(int64_t rows, float vf_coef, float *losses, void *workspace, cudaStream_t s);

// Workspace of the LM-head calls: header | per-row chunk partials of the forward call | row order [M] i32 |
// packed copy of H [M, K] bf16 (offsets in bytes from the workspace base; ppo_lmhead_workspace_bytes = bytes)
struct LmWorkspace {
    size_t order_off, packed_off, bytes;
};
LmWorkspace lm_workspace(int64_t M, int64_t K, int64_t V);
// Rows with mask 1 of H [M, K] packed, in row order, into the workspace's copy; their number goes to the header's
// n_tokens, their original indices to the order array (the other rows' indices follow). The copy's rows from that
// number up to the next multiple of 128 (or M) are zero-filled, so that a contraction over the packed rows may run
// over whole blocks.
int launch_lm_pack_rows(const void *H, int64_t M, int64_t K, const uint8_t *mask, void *workspace,
                        const LmWorkspace &lay, cudaStream_t s);

// tuning options (ppo_set_option)
int option_value(int key);

}   // namespace ppo
