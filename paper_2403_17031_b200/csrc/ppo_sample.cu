// Temperature sampling fused into the log-prob / entropy pass (the step before step 1: Table "PPO
// hyperparameters", temperature 0.7): one kernel draws the token of every row from
// softmax(logits / tau) and returns its log-prob, the row's entropy and log-sum-exp, so the logits are
// streamed from HBM once for both.
//
// The draw is defined so that it can be reproduced on a CPU token by token:
//   * Philox4x32-10 (counter-based; Salmon et al., SC'11): key = seed, counter = (j / 4, row, offset low,
//     offset high), word j % 4 belongs to element j of the row;
//   * u_j = (floor(word / 2^9) + 1/2) * 2^-23, an fp32 number strictly inside (0, 1);
//   * the token is the j that minimises E_j / 2^(y_j) with E_j = -log2(u_j) (an exponential race; the
//     same as the Gumbel-max rule argmax_j [y_j - log2(-log2 u_j)]), y_j = logit_j * log2(e) / tau.
//     Candidates are compared by cross-multiplication (E_j * e_best < E_best * e_j with e = 2^(y - max)),
//     so the race costs no division and reuses the exponential that the softmax sums need anyway;
//     exact ties go to the lowest index.
// One block per row, one pass: the exponentials are taken relative to the maximum of the row's first pack
// (any reference serves the race and the sums); a row whose sums overflow that way, or that holds a NaN or
// an infinity, is repeated with its exact maximum. The generator dominates: ~10 integer instructions per
// logit next to ~12 for everything else, so this kernel is bound by instruction issue, not by HBM.
#include "ppo_rows.cuh"

namespace ppo {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;

// the ten round keys depend on the seed only: computed once per thread (uniform across the grid)
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
    __device__ __forceinline__ void init(uint32_t a, uint32_t b)
    {
#pragma unroll
        for (int r = 0; r < 10; ++r) {
            k0[r] = a + (uint32_t)r * kPhiloxW0;
            k1[r] = b + (uint32_t)r * kPhiloxW1;
        }
    }
};

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys &k,
                                              uint32_t (&o)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;   // one wide multiply each
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.k0[r];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.k1[r];
        c3 = (uint32_t)p0;
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

struct SampleSmem {
    float rs[32], ru[32], re[32], rl[32];
    int rj[32];
    float bs, bu;
    int redo;
};

// softmax sums and race of one row relative to the reference m (base-2 units); result in thread 0
template <typename T, bool VECTOR, int THREADS>
__device__ __forceinline__ void sums_and_race(const T *src, int V, float c, float m, uint32_t row, const SampleArgs &a,
                                              const PhiloxKeys &keys, SampleSmem &sm, float &s_out, float &u_out,
                                              Race &best_out)
{
    constexpr int N = Pack<T>::N;
    constexpr int WARPS = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float nm = -m;
    float s0 = 0.f, s1 = 0.f, u0 = 0.f, u1 = 0.f;
    Race best;
    best.init();
    if (VECTOR) {
        const uint4 *src4 = reinterpret_cast<const uint4 *>(src);
        const int nvec = V / N;
        for (int i = threadIdx.x; i < nvec; i += THREADS) {
            float x[N];
            Pack<T>::unpack_clamped(src4[i], x);
#pragma unroll
            for (int h = 0; h < N / 4; ++h) {
                uint32_t w[4];
                philox4x32_10((uint32_t)(i * (N / 4) + h), row, a.off_lo, a.off_hi, keys, w);
#pragma unroll
                for (int q = 0; q < 4; q += 2) {   // packed fp32x2 arithmetic: two elements per instruction
                    const float2 t = __ffma2_rn(make_float2(x[h * 4 + q], x[h * 4 + q + 1]), make_float2(c, c),
                                                make_float2(nm, nm));
                    const float2 e = make_float2(ex2(t.x), ex2(t.y));
                    const float2 sn = __fadd2_rn(make_float2(s0, s1), e);
                    const float2 un = __ffma2_rn(e, t, make_float2(u0, u1));
                    s0 = sn.x; s1 = sn.y; u0 = un.x; u1 = un.y;
                    best.offer(e.x, log2_uniform(w[q]), i * N + h * 4 + q);
                    best.offer(e.y, log2_uniform(w[q + 1]), i * N + h * 4 + q + 1);
                }
            }
        }
    } else {
        for (int j = threadIdx.x; j < V; j += THREADS) {
            float x = Pack<T>::load1(src + j);
            x = (x != x) ? x : fmaxf(x, kNegBig);
            uint32_t w[4];
            philox4x32_10((uint32_t)(j >> 2), row, a.off_lo, a.off_hi, keys, w);
            const float t = fmaf(x, c, nm);
            const float e = ex2(t);
            s0 += e;
            u0 = fmaf(e, t, u0);
            best.offer(e, log2_uniform(w[j & 3]), j);
        }
    }
    // block merge: sums by addition, race by comparison (fixed order: lanes, then warps)
    float s = s0 + s1, u = u0 + u1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, off);
        u += __shfl_xor_sync(0xffffffffu, u, off);
        Race o;
        o.e = __shfl_xor_sync(0xffffffffu, best.e, off);
        o.L = __shfl_xor_sync(0xffffffffu, best.L, off);
        o.j = __shfl_xor_sync(0xffffffffu, best.j, off);
        best.merge(o);
    }
    __syncthreads();   // the arrays below may still be read from an earlier call
    if (lane == 0) {
        sm.rs[warp] = s; sm.ru[warp] = u; sm.re[warp] = best.e; sm.rl[warp] = best.L; sm.rj[warp] = best.j;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        s = 0.f; u = 0.f;
        best.init();
        for (int w = 0; w < WARPS; ++w) {
            s += sm.rs[w]; u += sm.ru[w];
            Race o;
            o.e = sm.re[w]; o.L = sm.rl[w]; o.j = sm.rj[w];
            best.merge(o);
        }
    }
    s_out = s; u_out = u; best_out = best;
}

template <typename T, bool VECTOR, int THREADS>
__global__ void __launch_bounds__(THREADS)
sample_kernel(const SampleArgs a)
{
    constexpr int N = Pack<T>::N;
    constexpr int WARPS = THREADS / 32;
    __shared__ SampleSmem sm;
    const int64_t row = blockIdx.x;
    const T *src = reinterpret_cast<const T *>(a.logits) + row * a.row_stride;
    const int V = a.V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    PhiloxKeys keys;
    keys.init(a.k0, a.k1);

    // First attempt with the maximum of the row's first pack as the reference of the exponentials (any
    // reference works for the race and the sums as long as nothing overflows): one pass over the row.
    float m = VECTOR ? row_reference<T>(src, a.c) : safe_reference(fmaxf(Pack<T>::load1(src), kNegBig), a.c);
    float s, u;
    Race best;
    sums_and_race<T, VECTOR, THREADS>(src, V, a.c, m, (uint32_t)row, a, keys, sm, s, u, best);
    if (threadIdx.x == 0) sm.redo = !(s < 1.0e37f) || !(fabsf(u) < 1.0e37f);
    __syncthreads();
    if (sm.redo) {
        // a sum overflowed (an element lies more than ~2^127 above the reference) or the row holds a NaN or
        // +inf: take the exact maximum (NaN-blind; a NaN then shows up in the sums again) and repeat
        float mx = kNegBig;
        if (VECTOR) {
            const uint4 *src4 = reinterpret_cast<const uint4 *>(src);
            const int nvec = V / N;
            for (int i = threadIdx.x; i < nvec; i += THREADS) {
                float x[N], xm;
                Pack<T>::unpack(src4[i], x, xm);
                mx = fmaxf(mx, xm);
            }
        } else {
            for (int j = threadIdx.x; j < V; j += THREADS) mx = fmaxf(mx, fmaxf(Pack<T>::load1(src + j), kNegBig));
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
        sums_and_race<T, VECTOR, THREADS>(src, V, a.c, m, (uint32_t)row, a, keys, sm, s, u, best);
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
    constexpr int THREADS = 256;
    const int n = dtype == PPO_F32 ? 4 : 8;
    const bool vec = aligned16(logits) && (row_stride * es) % 16 == 0 && V % n == 0;
    const unsigned grid = (unsigned)rows;
    if (dtype == PPO_F32) {
        if (vec) sample_kernel<float, true, THREADS><<<grid, THREADS, 0, s>>>(a);
        else sample_kernel<float, false, THREADS><<<grid, THREADS, 0, s>>>(a);
    } else {
        if (vec) sample_kernel<__nv_bfloat16, true, THREADS><<<grid, THREADS, 0, s>>>(a);
        else sample_kernel<__nv_bfloat16, false, THREADS><<<grid, THREADS, 0, s>>>(a);
    }
    return launch_status();
}
