// Temperature sampling fused into the log-prob / entropy pass (the step before step 1: Table "PPO
// hyperparameters", temperature 0.7): one kernel draws the token of every row from
// softmax(logits / tau) and returns its log-prob, the row's entropy and log-sum-exp, so the logits are
// streamed from HBM once for both.
//
// The draw is defined so that it can be reproduced on a CPU token by token:
//   * Philox4x32-10 (counter-based; Salmon et al., SC'11), key = seed; a 32-bit word w gives the uniform
//     (floor(w / 2^9) + 1/2) * 2^-23, an fp32 number strictly inside (0, 1);
//   * an exponential race (the Gumbel-max rule) in two levels. The row is dealt into 256 classes in runs of 8
//     elements, class(j) = (j / 8) mod 256, which is exactly the set of elements thread c of a 256-thread block
//     streams. Level 1: class c has weight W_c = sum of 2^(y_j) over its elements (y_j = logit_j * log2(e) / tau:
//     the thread's share of the softmax sum, needed anyway) and the uniform of word c % 4 of the counter
//     (2^31 + c / 4, row, offset low, offset high); the class that minimises -log2(v_c) / W_c wins. Level 2: inside
//     that class, element j has the uniform of word j % 4 of the counter (j / 4, row, offset low, offset high) and
//     the element that minimises -log2(u_j) / 2^(y_j) is the token. Every element is drawn with probability
//     softmax(logits / tau)_j, and only 256 + V / 256 uniforms per row are ever needed, so the generator costs
//     nothing next to the stream of logits: the kernel runs at the speed of the plain log-prob pass.
//     Candidates are compared by cross-multiplication (E_a * w_b < E_b * w_a), no division; exact ties go to
//     the lowest index.
// One block of 256 threads per row, one pass over the logits: the exponentials are taken relative to the maximum
// of the row's first pack (any reference serves the race and the sums); a row whose sums overflow that way, or
// that holds a NaN or an infinity (-inf included), is repeated with clamped values and its exact maximum. Then two short block-wide steps: the race
// between the 256 class sums, and the race between the members of the winning class (one member per thread,
// re-read from L2).
#include "ppo_rows.cuh"

namespace ppo {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;

// (the round keys are derived on the fly: a thread runs the generator twice per row, and nothing of it should
// occupy registers during the pass over the logits)
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&o)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;   // one wide multiply each
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c3 = (uint32_t)p0;
        k0 += kPhiloxW0;
        k1 += kPhiloxW1;
    }
    o[0] = c0; o[1] = c1; o[2] = c2; o[3] = c3;
}

// 32-bit word -> log2(u) < 0, u = (word >> 9 + 1/2) * 2^-23 (built in the mantissa: no int->float convert).
// The exponential variate of the race is E = -log2(u); the sign stays folded into the comparisons.
__device__ __forceinline__ float log2_uniform(uint32_t w)
{
    const float u = __uint_as_float(0x3f800000u | (w >> 9)) - 0.99999994f;   // 1 + k 2^-23 - (1 - 2^-24): exact
    float l;
    asm("lg2.approx.f32 %0, %1;" : "=f"(l) : "f"(u));
    return l;
}

struct Race {
    float e, L;   // best candidate so far: e = 2^(y - reference), L = log2(u) = -E
    int j;
    __device__ __forceinline__ void init() { e = 0.f; L = -1.f; j = 0x7fffffff; }
    // candidate (e1, L1) beats the best when E1 / e1 < E / e, i.e. L1 * e > L * e1 (both sides <= 0);
    // offered in increasing index order, so a strict comparison leaves ties with the lowest index
    __device__ __forceinline__ void offer(float e1, float L1, int j1)
    {
        const float2 pr = __fmul2_rn(make_float2(L1, L), make_float2(e, e1));   // both products in one instruction
        if (pr.x > pr.y) { e = e1; L = L1; j = j1; }
    }
    __device__ __forceinline__ void merge(const Race &o)
    {
        const float l = o.L * e, r = L * o.e;
        if (l > r || (l == r && o.j < j)) *this = o;
    }
};

struct SampleArgs {
    const void *logits;
    int V;
    int64_t row_stride;
    float c;
    uint32_t k0, k1, off_lo, off_hi;
    int32_t *tokens;
    float *logprob, *entropy, *lse;
    int *status;
};

constexpr int kSampleThreads = 256;      // = number of classes of the draw
constexpr int kRun = 8;                  // consecutive elements that go to the same class
constexpr uint32_t kClassCounterBase = 0x80000000u;

struct SampleSmem {
    float rs[8], ru[8], re[8], rl[8];
    int rj[8];
    float bs, bu, be;
    int bj;
    int redo;
};

// block-wide race (fixed order: lanes, then warps); the winner is returned to every thread
__device__ __forceinline__ Race block_race(Race best, SampleSmem &sm)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Race o;
        o.e = __shfl_xor_sync(0xffffffffu, best.e, off);
        o.L = __shfl_xor_sync(0xffffffffu, best.L, off);
        o.j = __shfl_xor_sync(0xffffffffu, best.j, off);
        best.merge(o);
    }
    __syncthreads();   // the arrays below may still be read from the step before
    if (lane == 0) { sm.re[warp] = best.e; sm.rl[warp] = best.L; sm.rj[warp] = best.j; }
    __syncthreads();
    Race w;
    w.init();
#pragma unroll
    for (int k = 0; k < kSampleThreads / 32; ++k) {
        Race o;
        o.e = sm.re[k]; o.L = sm.rl[k]; o.j = sm.rj[k];
        w.merge(o);
    }
    return w;
}

// The softmax sums of one row relative to the reference m (base-2 units), thread c summing class c, then the two
// levels of the race. Returns the row sums (s, u) and the winning element to every thread.
// CLAMP: -inf logits are clamped (first attempt without: 0 * -inf then turns the entropy sum into NaN and the row is repeated).
template <typename T, bool VECTOR, bool CLAMP>
__device__ __forceinline__ void sums_and_race(const T *src, int V, float c, float m, uint32_t row, const SampleArgs &a,
                                              SampleSmem &sm, float &s_out, float &u_out, Race &best_out)
{
    constexpr int N = Pack<T>::N, PPR = kRun / N;   // packs per run: 1 (bf16) or 2 (fp32)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float nm = -m;
    const int n_runs = (V + kRun - 1) / kRun;
    FixedAcc acc;
    acc.init();
    if (VECTOR) {
        const uint4 *src4 = reinterpret_cast<const uint4 *>(src);
        const int nvec = V / N;
        constexpr int UNROLL = 4 / PPR;             // four 16-byte loads in flight per thread
        int g = threadIdx.x;
        for (; g + (UNROLL - 1) * kSampleThreads < n_runs; g += UNROLL * kSampleThreads) {
            uint4 v[UNROLL][PPR];
            bool have[UNROLL][PPR];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
#pragma unroll
                for (int h = 0; h < PPR; ++h) {
                    const int i = (g + k * kSampleThreads) * PPR + h;
                    have[k][h] = i < nvec;       // (fp32 with V % 8 == 4: the last run is half a run)
                    if (have[k][h]) v[k][h] = ld_stream(src4 + i);
                }
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
#pragma unroll
                for (int h = 0; h < PPR; ++h)
                    if (have[k][h]) accumulate_fixed<T, true, CLAMP>(v[k][h], c, nm, acc);
        }
        for (; g < n_runs; g += kSampleThreads)
#pragma unroll
            for (int h = 0; h < PPR; ++h) {
                const int i = g * PPR + h;
                if (i < nvec) accumulate_fixed<T, true, CLAMP>(ld_stream(src4 + i), c, nm, acc);
            }
    } else {
        for (int g = threadIdx.x; g < n_runs; g += kSampleThreads)
            for (int q = 0; q < kRun; ++q) {
                const int j = g * kRun + q;
                if (j >= V) break;
                float x = Pack<T>::load1(src + j);
                x = (x != x) ? x : fmaxf(x, kNegBig);
                const float t = fmaf(x, c, nm);
                const float e = ex2(t);
                acc.s0 += e;
                acc.u0 = fmaf(e, t, acc.u0);
            }
    }
    // ---- level 1: the class sums race with one uniform each; the row sums are merged on the way
    const float W = acc.s0 + acc.s1;
    float s = W, u = acc.u0 + acc.u1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, off);
        u += __shfl_xor_sync(0xffffffffu, u, off);
    }
    __syncthreads();
    if (lane == 0) { sm.rs[warp] = s; sm.ru[warp] = u; }
    uint32_t w[4];
    philox4x32_10(kClassCounterBase + (threadIdx.x >> 2), row, a.off_lo, a.off_hi, a.k0, a.k1, w);
    Race cls;
    cls.e = W;
    cls.L = log2_uniform(w[threadIdx.x & 3]);
    cls.j = (int)threadIdx.x;
    if (!(W > 0.f)) cls.init();                 // a class without weight (or with a NaN) never wins
    cls = block_race(cls, sm);                  // (its barriers also publish rs / ru)
    s = 0.f; u = 0.f;
#pragma unroll
    for (int k = 0; k < kSampleThreads / 32; ++k) { s += sm.rs[k]; u += sm.ru[k]; }
    // ---- level 2: the members of the winning class race, one member per thread
    Race best;
    best.init();
    if (cls.j != 0x7fffffff) {
        const int c_star = cls.j;
        for (int q = threadIdx.x;; q += kSampleThreads) {
            const int run = c_star + (q / kRun) * kSampleThreads;
            if (run >= n_runs) break;
            const int j = run * kRun + (q % kRun);
            if (j < V) {
                float x = Pack<T>::load1(src + j);
                x = (x != x) ? x : fmaxf(x, kNegBig);
                const float e = ex2(fmaf(x, c, nm));
                philox4x32_10((uint32_t)(j >> 2), row, a.off_lo, a.off_hi, a.k0, a.k1, w);
                const uint32_t wj = (j & 2) ? ((j & 1) ? w[3] : w[2]) : ((j & 1) ? w[1] : w[0]);
                if (e > 0.f) best.offer(e, log2_uniform(wj), j);
            }
        }
    }
    best = block_race(best, sm);
    s_out = s; u_out = u; best_out = best;
}

template <typename T, bool VECTOR>
__global__ void __launch_bounds__(kSampleThreads, 8)
sample_kernel(const SampleArgs a)
{
    constexpr int N = Pack<T>::N;
    constexpr int WARPS = kSampleThreads / 32;
    __shared__ SampleSmem sm;
    const int64_t row = blockIdx.x;
    const T *src = reinterpret_cast<const T *>(a.logits) + row * a.row_stride;
    const int V = a.V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // First attempt with the maximum of the row's first pack as the reference of the exponentials (any
    // reference works for the race and the sums as long as nothing overflows): one pass over the row.
    float m = VECTOR ? row_reference<T>(src, a.c) : safe_reference(fmaxf(Pack<T>::load1(src), kNegBig), a.c);
    float s, u;
    Race best;
    sums_and_race<T, VECTOR, false>(src, V, a.c, m, (uint32_t)row, a, sm, s, u, best);
    if (!(s < 1.0e37f) || !(fabsf(u) < 1.0e37f)) {   // (s and u are the same in every thread)
        // a sum overflowed (an element lies more than ~2^127 above the reference) or the row holds a NaN or
        // +inf: take the exact maximum (NaN-blind; a NaN then shows up in the sums again) and repeat
        float mx = kNegBig;
        if (VECTOR) {
            const uint4 *src4 = reinterpret_cast<const uint4 *>(src);
            const int nvec = V / N;
            for (int i = threadIdx.x; i < nvec; i += kSampleThreads) {
                float x[N], xm;
                Pack<T>::unpack(src4[i], x, xm);
                mx = fmaxf(mx, xm);
            }
        } else {
            for (int j = threadIdx.x; j < V; j += kSampleThreads) mx = fmaxf(mx, fmaxf(Pack<T>::load1(src + j), kNegBig));
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        __syncthreads();
        if (lane == 0) sm.rs[warp] = mx;
        __syncthreads();
        mx = sm.rs[lane < WARPS ? lane : 0];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        m = safe_reference(mx, a.c);
        __syncthreads();
        sums_and_race<T, VECTOR, true>(src, V, a.c, m, (uint32_t)row, a, sm, s, u, best);
    }
    if (threadIdx.x == 0) {
        int tok = best.j;
        float lp, H, L;
        // a NaN or +inf in the row, or no element with non-zero probability: nothing is drawn
        if (!(s < 3.0e38f) || !(fabsf(u) < 3.0e38f) || tok == 0x7fffffff) {
            tok = -1;
            lp = H = L = __int_as_float(0x7fc00000);
            if (a.status) atomicOr(a.status, PPO_DEV_BAD_ROW);
        } else {
            float x = Pack<T>::load1(src + tok);          // the winner's own logit, for its log-prob
            x = fmaxf(x, kNegBig);
            const float l2s = log2f(s);
            lp = (fmaf(x, a.c, -m) - l2s) * kLn2;
            H = (l2s - u / s) * kLn2;
            L = (m + l2s) * kLn2;
        }
        a.tokens[row] = tok;
        if (a.logprob) a.logprob[row] = lp;
        if (a.entropy) a.entropy[row] = H;
        if (a.lse) a.lse[row] = L;
    }
}

}   // namespace ppo

using namespace ppo;

extern "C" int ppo_sample_logprob_entropy(const void *logits, int dtype, int64_t rows, int64_t V, int64_t row_stride,
                                          float temperature, uint64_t seed, uint64_t offset, int32_t *tokens_out,
                                          float *logprob, float *entropy, float *lse, void *workspace, void *stream)
{
    if (dtype != PPO_F32 && dtype != PPO_BF16) return PPO_ERR_DTYPE;
    if (rows < 0 || rows >= ((int64_t)1 << 31) || V <= 0 || V >= ((int64_t)1 << 31) || row_stride < V)
        return PPO_ERR_SHAPE;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    if (rows == 0) return PPO_OK;
    if (!logits || !tokens_out) return PPO_ERR_NULL;
    const size_t es = dtype == PPO_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return PPO_ERR_ALIGN;
    SampleArgs a;
    a.logits = logits;
    a.V = (int)V;
    a.row_stride = row_stride;
    a.c = kLog2e / temperature;
    a.k0 = (uint32_t)seed;
    a.k1 = (uint32_t)(seed >> 32);
    a.off_lo = (uint32_t)offset;
    a.off_hi = (uint32_t)(offset >> 32);
    a.tokens = tokens_out;
    a.logprob = logprob;
    a.entropy = entropy;
    a.lse = lse;
    a.status = workspace ? &ws_header(workspace)->status : nullptr;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int n = dtype == PPO_F32 ? 4 : 8;
    const bool vec = aligned16(logits) && (row_stride * es) % 16 == 0 && V % n == 0;
    const unsigned grid = (unsigned)rows;
    if (dtype == PPO_F32) {
        if (vec) sample_kernel<float, true><<<grid, kSampleThreads, 0, s>>>(a);
        else sample_kernel<float, false><<<grid, kSampleThreads, 0, s>>>(a);
    } else {
        if (vec) sample_kernel<__nv_bfloat16, true><<<grid, kSampleThreads, 0, s>>>(a);
        else sample_kernel<__nv_bfloat16, false><<<grid, kSampleThreads, 0, s>>>(a);
    }
    return launch_status();
}
