// Device code shared by the row kernels: 16-byte element packs, the softmax accumulators and the
// statistics pass over one row.
#pragma once

#include "ppo_common.cuh"

namespace ppo {

// ---------------------------------------------------------------- element packs
// A "pack" is one 16-byte vector: 8 bf16 or 4 fp32 logits.
template <typename T> struct Pack;

template <> struct Pack<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ float clampf(float x) { return (x != x) ? x : fmaxf(x, kNegBig); }
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&x)[4], float &xmax)
    {
        // fmaxf drops NaN; clampf keeps it so a NaN logit poisons the row as documented
        x[0] = clampf(__uint_as_float(v.x));
        x[1] = clampf(__uint_as_float(v.y));
        x[2] = clampf(__uint_as_float(v.z));
        x[3] = clampf(__uint_as_float(v.w));
        xmax = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    }
    static __device__ __forceinline__ void unpack_clamped(const uint4 &v, float (&x)[4])
    {
        x[0] = clampf(__uint_as_float(v.x));
        x[1] = clampf(__uint_as_float(v.y));
        x[2] = clampf(__uint_as_float(v.z));
        x[3] = clampf(__uint_as_float(v.w));
    }
    static __device__ __forceinline__ void unpack_raw(const uint4 &v, float (&x)[4])
    {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&d)[4])
    {
        return make_uint4(__float_as_uint(d[0]), __float_as_uint(d[1]), __float_as_uint(d[2]),
                          __float_as_uint(d[3]));
    }
    static __device__ __forceinline__ float load1(const float *p) { return *p; }
    static __device__ __forceinline__ void store1(float *p, float v) { *p = v; }
};

template <> struct Pack<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ __nv_bfloat162 as2(uint32_t w)
    {
        return *reinterpret_cast<__nv_bfloat162 *>(&w);
    }
    static __device__ __forceinline__ uint32_t bits(__nv_bfloat162 h) { return *reinterpret_cast<uint32_t *>(&h); }
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&x)[8], float &xmax)
    {
        const __nv_bfloat162 lim = __float2bfloat162_rn(kNegBig);
        const __nv_bfloat162 h0 = __hmax2_nan(as2(v.x), lim), h1 = __hmax2_nan(as2(v.y), lim),
                             h2 = __hmax2_nan(as2(v.z), lim), h3 = __hmax2_nan(as2(v.w), lim);
        const uint32_t wm = bits(__hmax2(__hmax2(h0, h1), __hmax2(h2, h3)));
        xmax = fmaxf(__uint_as_float(wm << 16), __uint_as_float(wm & 0xffff0000u));
        widen(bits(h0), bits(h1), bits(h2), bits(h3), x);
    }
    // bf16 -> fp32 is a 16-bit shift of the bit pattern (plain integer ops, no convert unit)
    static __device__ __forceinline__ void widen(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, float (&x)[8])
    {
        x[0] = __uint_as_float(w0 << 16); x[1] = __uint_as_float(w0 & 0xffff0000u);
        x[2] = __uint_as_float(w1 << 16); x[3] = __uint_as_float(w1 & 0xffff0000u);
        x[4] = __uint_as_float(w2 << 16); x[5] = __uint_as_float(w2 & 0xffff0000u);
        x[6] = __uint_as_float(w3 << 16); x[7] = __uint_as_float(w3 & 0xffff0000u);
    }
    // clamped at kNegBig (NaN kept) but without the pack maximum
    static __device__ __forceinline__ void unpack_clamped(const uint4 &v, float (&x)[8])
    {
        const __nv_bfloat162 lim = __float2bfloat162_rn(kNegBig);
        widen(bits(__hmax2_nan(as2(v.x), lim)), bits(__hmax2_nan(as2(v.y), lim)), bits(__hmax2_nan(as2(v.z), lim)),
              bits(__hmax2_nan(as2(v.w), lim)), x);
    }
    static __device__ __forceinline__ void unpack_raw(const uint4 &v, float (&x)[8]) { widen(v.x, v.y, v.z, v.w, x); }
    static __device__ __forceinline__ uint4 pack(const float (&d)[8])
    {
        return make_uint4(bits(__floats2bfloat162_rn(d[0], d[1])), bits(__floats2bfloat162_rn(d[2], d[3])),
                          bits(__floats2bfloat162_rn(d[4], d[5])), bits(__floats2bfloat162_rn(d[6], d[7])));
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
};

// streaming 16-byte global accesses (data is touched once: evict-first)
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) { __stcs(p, v); }

// fold one pack into the running state, moving the reference up when the pack exceeds it
template <typename T>
__device__ __forceinline__ void accumulate_online(const uint4 &v, float c, SoftmaxState &st)
{
    float x[Pack<T>::N], xmax;
    Pack<T>::unpack(v, x, xmax);
    const float ymax = xmax * c;
    if (ymax > st.m) st.rebase(ymax);
    const float nm = -st.m;
#pragma unroll
    for (int k = 0; k < Pack<T>::N; ++k) st.add(fmaf(x[k], c, nm));
}

// Reference (base-2 units) taken from a pack maximum. A pack that holds only -inf (clamped to
// kNegBig) must not become the reference: at that magnitude x*c - ref no longer cancels exactly.
__device__ __forceinline__ float safe_reference(float xmax, float c) { return xmax > -1.0e29f ? xmax * c : 0.f; }

// Two independent accumulator pairs relative to a FIXED reference (nm = -reference).
struct FixedAcc {
    float s0, u0, s1, u1;
    __device__ __forceinline__ void init() { s0 = u0 = s1 = u1 = 0.f; }
};

// CLAMP = false is the fast path: a -inf logit then gives 0 * -inf = NaN in the entropy sum, which
// the caller detects after the fact and repairs by redoing the packs with CLAMP = true.
template <typename T, bool ENTROPY, bool CLAMP = false>
__device__ __forceinline__ void accumulate_fixed(const uint4 &v, float c, float nm, FixedAcc &a)
{
    float x[Pack<T>::N];
    if (CLAMP) Pack<T>::unpack_clamped(v, x);
    else Pack<T>::unpack_raw(v, x);
    // packed fp32x2 instructions (sm_100): two multiply-adds or adds per issue slot, each lane rounded like the
    // scalar instruction - same sums, fewer instructions (and less power) around the exponentials
    const float2 cc = make_float2(c, c), nn = make_float2(nm, nm);
    float2 s = make_float2(a.s0, a.s1), u = make_float2(a.u0, a.u1);
#pragma unroll
    for (int k = 0; k < Pack<T>::N; k += 2) {
        const float2 t = __ffma2_rn(make_float2(x[k], x[k + 1]), cc, nn);
        const float2 e = make_float2(ex2(t.x), ex2(t.y));
        s = __fadd2_rn(s, e);
        if (ENTROPY) u = __ffma2_rn(e, t, u);
    }
    a.s0 = s.x; a.s1 = s.y;
    a.u0 = u.x; a.u1 = u.y;
}

// Statistics pass over one row. VECTOR: 16-byte packs (row base 16-byte aligned, V % N == 0);
// otherwise element by element. STAGE: also park the raw packs / elements in shared memory.
//
// Fast path: the softmax sums do not need the exact maximum as reference, only one that keeps
// 2^(y - ref) inside fp32 range. Every thread of the row uses the same fixed reference m_common
// (see row_reference) and never moves it, which removes the per-pack maximum, compare and rescale
// from the inner loop and lets the block merge its threads by plain addition. If a later element exceeds the reference by more than ~2^127 the sum overflows to
// inf, and a -inf logit turns the entropy sum into NaN (0 * -inf); both are detected after the loop
// and the thread redoes its packs with the clamped online update.
// Common reference of a row for the vector path: the maximum of the row's first pack (every thread
// reads the same 16 bytes), in base-2 units.
template <typename T>
__device__ __forceinline__ float row_reference(const T *__restrict__ src, float c)
{
    float x[Pack<T>::N], xmax;
    Pack<T>::unpack(*reinterpret_cast<const uint4 *>(src), x, xmax);
    return safe_reference(xmax, c);
}

template <typename T, bool VECTOR, bool STAGE, bool ENTROPY, int THREADS, int UNROLL>
__device__ __forceinline__ SoftmaxState row_statistics(const T *__restrict__ src, int V, float c, void *stage,
                                                       float m_common)
{
    SoftmaxState st;
    st.init();
    if (VECTOR) {
        constexpr int N = Pack<T>::N;
        const uint4 *src4 = reinterpret_cast<const uint4 *>(src);
        uint4 *stage4 = reinterpret_cast<uint4 *>(stage);
        const int nvec = V / N;
        int i = threadIdx.x;
        if (i < nvec) {
            FixedAcc acc;
            acc.init();
            uint4 v[UNROLL];
            // first group: also fixes the reference
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
                if (i + k * THREADS < nvec) v[k] = ld_stream(src4 + i + k * THREADS);
            st.m = m_common;
            const float nm = -st.m;
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
                if (i + k * THREADS < nvec) {
                    if (STAGE) stage4[i + k * THREADS] = v[k];
                    accumulate_fixed<T, ENTROPY>(v[k], c, nm, acc);
                }
            i += UNROLL * THREADS;
            for (; i + (UNROLL - 1) * THREADS < nvec; i += UNROLL * THREADS) {
#pragma unroll
                for (int k = 0; k < UNROLL; ++k) v[k] = ld_stream(src4 + i + k * THREADS);
#pragma unroll
                for (int k = 0; k < UNROLL; ++k) {
                    if (STAGE) stage4[i + k * THREADS] = v[k];
                    accumulate_fixed<T, ENTROPY>(v[k], c, nm, acc);
                }
            }
            for (; i < nvec; i += THREADS) {
                const uint4 v1 = ld_stream(src4 + i);
                if (STAGE) stage4[i] = v1;
                accumulate_fixed<T, ENTROPY>(v1, c, nm, acc);
            }
            st.s = acc.s0 + acc.s1;
            st.u = acc.u0 + acc.u1;
            if (!(st.s < 1.0e37f) || !(fabsf(st.u) < 1.0e37f)) {
                // overflow (or NaN input): redo this thread's packs with a moving reference
                st.init();
                for (i = threadIdx.x; i < nvec; i += THREADS)
                    accumulate_online<T>(STAGE ? stage4[i] : src4[i], c, st);
                if (!ENTROPY) st.u = 0.f;
            }
        }
    } else {
        T *stage1 = reinterpret_cast<T *>(stage);
        for (int j = threadIdx.x; j < V; j += THREADS) {
            const T raw = src[j];
            if (STAGE) stage1[j] = raw;
            float x = Pack<T>::load1(&raw);
            x = (x != x) ? x : fmaxf(x, kNegBig);
            const float y = x * c;
            if (y > st.m) st.rebase(y);
            st.add(fmaf(x, c, -st.m));
        }
    }
    return st;
}

// ---------------------------------------------------------------- step 6 arguments
struct LossArgs {
    const void *logits;
    void *dlogits;
    int64_t rows;
    int V;
    const int32_t *tokens;
    const uint8_t *mask;
    const float *old_logprob, *advantages, *values_new, *values_old, *returns;
    // log-prob backward only (ppo_logprob_bwd): the gradient on each token's log-prob is given; the five
    // PPO inputs above and dvalues are null, and no loss term is computed
    const float *g_ext;
    float *dvalues, *new_logprob, *entropy, *dlogprob;
    float *partials;
    const int *n_tokens;
    int *status;
    float c;        // log2(e) / temperature
    float inv_tau;  // 1 / temperature
    float eps, eps_v, c1;
};

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// bulk-copy row engine (ppo_rows_bulk.cu); each returns PPO_ERR_UNSUPPORTED when the shape does
// not fit it, and the caller then takes the direct-load kernels
int launch_logprob_bulk(const void *logits, int dtype, int64_t rows, int V, int64_t row_stride,
                        const int32_t *tokens, const uint8_t *mask, float c, float *logprob, float *entropy,
                        float *lse, int *status, cudaStream_t s);
// (the engine's loss kernel also reduces the partials and writes `losses` itself)
// `dependent`: launch so that the kernel may start while the kernel before it in the stream still runs (it
// waits for the workspace header's flags before it reads that kernel's results)
// `reuse`: no prologue ran for this call; the kernel checks that the order in the workspace was built from this
// call's mask (PPO_DEV_BAD_REUSE and nothing written otherwise)
// `keep_back`: leave a few masked rows per block to the blocks that run out of real rows (calls that do not overlap
// a long producer kernel)
int launch_loss_bulk(const LossArgs &a, int dtype, void *workspace, float *losses, float vf_coef, bool dependent,
                     cudaStream_t s, bool reuse = false, bool keep_back = false);

}   // namespace ppo
