// Row engine: persistent thread blocks that stream whole logits rows through shared memory with
// bulk asynchronous copies (cp.async.bulk, completion counted on mbarriers).
//
//   * one producer thread per block issues the copies, 16 KB chunk by chunk, into a shared-memory
//     buffer that holds exactly one row; 16 consumer warps read the chunks from shared memory;
//   * every chunk has a "full" barrier (bytes have landed) and an "empty" barrier (all consumer
//     warps are done with it). A chunk is released as soon as its last reader is done, so the
//     next row's bytes stream in behind the pass that is still consuming the current row: the
//     block never drains its loads at a row boundary;
//   * step 1 (log-prob/entropy) makes one pass and releases chunks as it goes; step 6 (loss)
//     keeps the row for a second pass that writes the gradient IN PLACE over the logits in shared
//     memory; the producer ships each finished chunk with one bulk shared->global copy and refills
//     the space, one chunk behind, with the next row. Rows whose mask is 0 are only zero-filled: a
//     filler thread per block takes them from a shared work counter and writes them with bulk
//     shared->global copies of a small block of zeros while the consumers work on real rows (the
//     real-row phase alone leaves HBM bandwidth idle); consumers that run out of real rows join in (a
//     stand-alone call keeps a few masked rows per block back for them, so that the end of the kernel stays busy);
//   * step 6 hands its rows out dynamically (a counter in the workspace header; the row index reaches
//     the consumers through a small ring in shared memory), since SMs do not stream at equal speed;
//   * two blocks per SM while a row is <= 110 KB (bf16, V = 50304), one otherwise;
//   * step 6 may be launched while the kernel that produces its row order and advantages is still
//     running (programmatic dependent launch): it then polls two flags of the workspace header.
//
// Every wait is bounded: when it runs out the block records PPO_DEV_TIMEOUT in the status word. A block
// that never learns the row order (step 6 launched early) returns before anything is indexed through it,
// and block 0 writes NaN loss scalars; after any other run-out the block carries on with the same control
// flow (so no barrier is left short), which makes the outputs invalid but lets the kernel end, and the
// producer makes sure that none of its copies into shared memory is still in flight when the block retires.
#include "ppo_rows.cuh"

namespace ppo {

// CONS consumer threads per block (template parameter of everything below): 512 (16 warps) when two
// blocks share an SM, 960 (30 warps) when a row is so large that only one block fits. Derived sizes:
// CONS + 64 threads per block (+ one producer warp + one filler warp); two packs per consumer thread
// and chunk, i.e. chunks of CONS * 32 bytes (16 KB / 30 KB).
constexpr int kZeroBytes = 4096;                    // shared zeros, source of the bulk zero-fill stores
// A stand-alone loss call (its advantages are there from the start; a later PPO epoch finds the row order too) keeps
// this many masked rows per block (at most half of them) away from the filler threads. They are zero-filled by the
// consumer warps of blocks that have run out of real rows, so the last row time of the kernel, in which fewer and fewer
// blocks still hold a real row, is filled with finely divisible work (3.4% at B = 64, T = 53; nothing at large batches,
// where the amount is a small part of the masked rows). The call inside ppo_step, which overlaps the kernels that
// produce its advantages, keeps nothing back: there the fillers use the time in which the consumers still wait.
#ifndef PPO_REUSE_RESERVE_ROWS
#define PPO_REUSE_RESERVE_ROWS 3
#endif
constexpr int kReuseReserveRows = PPO_REUSE_RESERVE_ROWS;
constexpr int kMaxChunks = 14;                      // barriers provided per block
constexpr size_t kMaxRowBytes = 224 * 1024;         // the largest row one block can hold
#ifndef PPO_WAIT_TRIES
#define PPO_WAIT_TRIES (1u << 20)
#endif
constexpr uint32_t kWaitTries = PPO_WAIT_TRIES;     // x ~1 us per try (a test build makes the waits short)

struct EngineSmem {
    unsigned long long full[kMaxChunks];
    unsigned long long empty[kMaxChunks];
    float red[2][96];      // by row parity: a row's sums are read while the next row's are written
    int next_item;
    int is_last;
    int ring[4];           // row of the block's k-th item at [k % 4], -1 = no further item
    int n_tokens;          // step 6: number of mask==1 rows of the call
    int abort;             // step 6: the order that this call was told to reuse is not the one of its mask
    double lred[6 * 32];
    alignas(128) unsigned char zeros[kZeroBytes];
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(unsigned long long *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// Bounded wait for the phase with the given parity. Returns false (and sets the status bit) if
// the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, uint32_t parity, int *status)
{
    const uint32_t addr = smem_addr(bar);
    for (uint32_t it = 0; it < kWaitTries; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(ok)
            : "r"(addr), "r"(parity), "r"(1000u)
            : "memory");
        if (ok) return true;
    }
    if (status) atomicOr(status, PPO_DEV_TIMEOUT);
    return false;
}

// global -> shared bulk copy of `bytes` (multiple of 16; both addresses 16-byte aligned), read
// once: L2 evict-first
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, uint32_t bytes, unsigned long long *bar,
                                          uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

template <int CONS>
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"r"(CONS) : "memory"); }

// merge over the consumer warps (named barrier 1); result to every consumer thread
template <int CONS>
__device__ __forceinline__ SoftmaxState consumer_merge(SoftmaxState st, float *red, int ct)
{
    constexpr int kConsumerWarps = CONS / 32;
    st = warp_merge(st);
    const int lane = ct & 31, warp = ct >> 5;
    if (lane == 0) {
        red[warp] = st.m;
        red[32 + warp] = st.s;
        red[64 + warp] = st.u;
    }
    consumer_sync<CONS>();
    SoftmaxState t;
    if (lane < kConsumerWarps) {
        t.m = red[lane];
        t.s = red[32 + lane];
        t.u = red[64 + lane];
    } else {
        t.init();
    }
    st = warp_merge(t);
    consumer_sync<CONS>();
    return st;
}

// Merge for the common case in which no consumer thread moved its reference: plain addition and one
// named barrier, which also ORs the "my reference differs" flags. Result valid in consumer thread 0,
// or in every consumer thread when ALL is set (each then adds the 16 warp sums itself, in the same
// order). `red` (96 floats) must not be rewritten before the caller's next consumer-wide barrier.
template <bool ALL, int CONS>
__device__ __forceinline__ SoftmaxState consumer_merge_common(SoftmaxState st, float m_common, float *red, int ct)
{
    constexpr int kConsumerWarps = CONS / 32;
    const int lane = ct & 31, warp = ct >> 5;
    if (st.s == 0.f) st.m = m_common;
    const uint32_t differs = st.m != m_common;
    const float s = warp_sum_f(st.s), u = warp_sum_f(st.u);
    if (lane == 0) {
        red[warp] = s;
        red[32 + warp] = u;
    }
    uint32_t any;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 q, %1, 0;\n"
        "bar.red.or.pred p, 1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(any)
        : "r"(differs), "r"(CONS)
        : "memory");
    if (any) {
        consumer_sync<CONS>();
        return consumer_merge<CONS>(st, red, ct);
    }
    SoftmaxState r;
    r.m = m_common;
    r.s = 0.f;
    r.u = 0.f;
    if (ALL || ct == 0) {
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            r.s += red[w];
            r.u += red[32 + w];
        }
    }
    return r;
}

// The sums of one thread as two-wide fp32 vectors: even elements of a pack in .x, odd ones in .y. The
// packed fp32 instructions of sm_100 (two fused multiply-adds or adds per issue slot, each lane rounded
// like the scalar instruction) halve the issue slots of the arithmetic around the exponentials: fewer
// instructions for the same bytes, which matters for the clocks under the board's power cap.
struct PairAcc {
    float2 s, u;
    __device__ __forceinline__ void init() { s = u = make_float2(0.f, 0.f); }
};

template <typename T, bool ENTROPY, bool CLAMP = false>
__device__ __forceinline__ void accumulate_pairs(const uint4 &v, float c, float nm, PairAcc &a)
{
    float x[Pack<T>::N];
    if (CLAMP) Pack<T>::unpack_clamped(v, x);
    else Pack<T>::unpack_raw(v, x);
    const float2 cc = make_float2(c, c), nn = make_float2(nm, nm);
#pragma unroll
    for (int k = 0; k < Pack<T>::N; k += 2) {
        const float2 t = __ffma2_rn(make_float2(x[k], x[k + 1]), cc, nn);
        const float2 e = make_float2(ex2(t.x), ex2(t.y));
        a.s = __fadd2_rn(a.s, e);
        if (ENTROPY) a.u = __ffma2_rn(e, t, a.u);
    }
}

// per-thread statistics with a fixed reference (the same for all threads of the row: the maximum of
// the row's first pack) that is only moved when a chunk overflows
template <typename T, bool ENTROPY>
struct ThreadStats {
    float m;          // reference, base-2 units
    PairAcc acc;
    __device__ __forceinline__ void init(float m_common)
    {
        m = m_common;
        acc.init();
    }
    __device__ __forceinline__ void rebase(float nm)
    {
        const float d = m - nm, a = ex2(d);
        acc.u.x = a * fmaf(d, acc.s.x, acc.u.x);
        acc.u.y = a * fmaf(d, acc.s.y, acc.u.y);
        acc.s.x *= a;
        acc.s.y *= a;
        m = nm;
    }
    // the sums left fp32 range, or a -inf/NaN logit turned the entropy sum into NaN
    __device__ __forceinline__ bool broken() const
    {
        return !(acc.s.x + acc.s.y < 1.0e35f) || !(fabsf(acc.u.x + acc.u.y) < 1.0e35f);
    }
    // slow path for one pack: clamped values, reference moved up to the pack maximum when needed
    __device__ __forceinline__ void pack_safe(const uint4 &v, float c)
    {
        float x[Pack<T>::N], xm;
        Pack<T>::unpack(v, x, xm);
        const float nm = safe_reference(xm, c);
        if (nm > m) rebase(nm);
        accumulate_pairs<T, ENTROPY, true>(v, c, -m, acc);
    }
    // fold up to two packs of one chunk
    __device__ __forceinline__ void chunk(const uint4 &v0, bool h0, const uint4 &v1, bool h1, float c)
    {
        if (!h0) return;                      // h1 implies h0
        const PairAcc save = acc;
        accumulate_pairs<T, ENTROPY>(v0, c, -m, acc);
        if (h1) accumulate_pairs<T, ENTROPY>(v1, c, -m, acc);
        if (broken()) {
            // overflow, or -inf/NaN logits: redo the chunk with clamped values and a moving reference
            acc = save;
            pack_safe(v0, c);
            if (h1) pack_safe(v1, c);
        }
    }
    __device__ __forceinline__ SoftmaxState state() const
    {
        SoftmaxState st;
        st.m = m;
        st.s = acc.s.x + acc.s.y;
        st.u = ENTROPY ? acc.u.x + acc.u.y : 0.f;
        return st;
    }
};

struct EngineArgs {
    // step 1 (MODE 0)
    const void *logits;
    int64_t rows;
    int64_t row_stride;     // elements
    int V;
    const int32_t *tokens;
    const uint8_t *mask;    // MODE 0: nullable
    float c;
    float *logprob, *entropy, *lse;
    int *status;
    // step 6 (MODE 1)
    LossArgs loss;
    const int32_t *order;
    WorkspaceHeader *hdr;
    float *losses;
    float vf_coef;
    int wait_flags;         // the launch overlaps the kernel that produces order / advantages: poll the header's flags
    int reuse;              // no prologue ran for this call: the order in the workspace must be the one of this mask
    int fill_reserve_rows;  // masked rows per block that the filler threads leave to the consumers' zero-fill phase
};

// number of masked rows that the filler threads may take
__device__ __forceinline__ int64_t filler_share(int64_t n_masked, int reserve_rows)
{
    const int64_t keep = (int64_t)reserve_rows * gridDim.x;
    return n_masked - (keep < n_masked / 2 ? keep : n_masked / 2);
}

template <int CONS>
__device__ __forceinline__ void block_sync_all() { asm volatile("bar.sync 2, %0;" ::"r"(CONS + 64) : "memory"); }

// End of the loss kernel, reached by every thread of the block once its role is finished: the
// block takes a ticket; the block that draws the last one sums the per-token partials of the whole
// batch in a fixed order and writes the loss scalars (so no separate reduction launch is needed
// and the result does not depend on which block happens to be last).
template <int CONS>
__device__ __forceinline__ void engine_epilogue(const EngineArgs &a, EngineSmem &sm)
{
    block_sync_all<CONS>();                       // every partial of this block has been written
    if (threadIdx.x == 0) {
        __threadfence();
        const int ticket = atomicAdd(&a.hdr->done_blocks, 1);
        sm.is_last = ticket == (int)gridDim.x - 1;
    }
    block_sync_all<CONS>();
    if (!sm.is_last) return;
    __threadfence();
    reduce_loss_partials<CONS + 64>(a.loss.partials, a.loss.rows, sm.n_tokens, a.vf_coef, a.losses, sm.lred,
                                    (int)threadIdx.x, [] { block_sync_all<CONS>(); });
    // every block is past the work counters: leave them ready for a call that reuses this order
    if (threadIdx.x == 0) {
        a.hdr->masked_next = 0;
        a.hdr->masked_tail = 0;
        a.hdr->real_next = 0;
        a.hdr->done_blocks = 0;
    }
}

// sign flip of a packed gradient (both bf16 halves of each word, or each fp32 word)
template <typename T> __device__ __forceinline__ uint4 negate_pack(uint4 v)
{
    const uint32_t m = sizeof(T) == 2 ? 0x80008000u : 0x80000000u;
    return make_uint4(v.x ^ m, v.y ^ m, v.z ^ m, v.w ^ m);
}

// pass 2 of the loss for one thread's two packs of a chunk: d = -+ 2^(x*c + off), packed and stored
template <typename T, bool NEG, int CONS>
__device__ __forceinline__ void gradient_packs(const uint4 *buf, uint4 *dst4, int i0, int nvec, float c, float off)
{
    constexpr int kConsumers = CONS;
    // (dst4 is the shared-memory row itself in the loss kernel: the gradient replaces the logits in place)
    constexpr int N = Pack<T>::N;
    const float2 cc = make_float2(c, c), oo = make_float2(off, off);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int i = i0 + h * kConsumers;
        if (i < nvec) {
            float x[N], d[N];
            Pack<T>::unpack_raw(buf[i], x);
#pragma unroll
            for (int q = 0; q < N; q += 2) {
                const float2 t = __ffma2_rn(make_float2(x[q], x[q + 1]), cc, oo);
                d[q] = ex2(t.x);
                d[q + 1] = ex2(t.y);
            }
            const uint4 g = Pack<T>::pack(d);
            dst4[i] = NEG ? negate_pack<T>(g) : g;
        }
    }
}

// MODE 0: log-prob/entropy. MODE 1: loss forward + backward.
template <typename T, int MODE, bool ENTROPY, int MIN_BLOCKS, int CONS>
__global__ void __launch_bounds__(CONS + 64, MIN_BLOCKS)
row_engine_kernel(const EngineArgs a)
{
    constexpr int kConsumers = CONS, kConsumerWarps = CONS / 32, kEngineThreads = CONS + 64;
    constexpr int kChunkPacks = 2 * CONS, kChunkBytes = kChunkPacks * 16;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ EngineSmem sm;
    constexpr int N = Pack<T>::N;
    const int V = a.V;
    const int nvec = V / N;
    const int nch = (nvec + kChunkPacks - 1) / kChunkPacks;
    const T *logits = reinterpret_cast<const T *>(a.logits);
    const int64_t stride = MODE == 0 ? a.row_stride : (int64_t)V;
    int *status = a.status;

    if (threadIdx.x == 0) {
        for (int c = 0; c < nch; ++c) {
            mbar_init(&sm.full[c], 1);
            mbar_init(&sm.empty[c], kConsumerWarps);
        }
        for (int q = 0; q < 4; ++q) sm.ring[q] = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (MODE == 1) {
        for (int i = threadIdx.x; i < kZeroBytes / 16; i += kEngineThreads)
            reinterpret_cast<uint4 *>(sm.zeros)[i] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // zeros are read by bulk copies
    }
    // step 6 inside ppo_step: this kernel may have been launched while the token-level kernel is still at
    // work; everything above touched shared memory only, from here on it reads what that kernel publishes
    // (the first flag carries the token count)
    if (MODE == 1 && threadIdx.x == 0) {
        sm.abort = 0;
        if (a.reuse) {   // the order must have been built from this mask, for this many rows, at this place
            const unsigned long long *sig = a.hdr->order_sig;
            if (sig[0] != (unsigned long long)reinterpret_cast<uintptr_t>(a.mask) || sig[1] != (unsigned long long)a.rows ||
                sig[2] != (unsigned long long)reinterpret_cast<uintptr_t>(a.order)) {
                atomicOr(status, PPO_DEV_BAD_REUSE);
                sm.abort = 1;
            }
        }
        if (a.wait_flags) {
            // a wait that ran out: nobody may have written the row order, so nothing may be indexed through it
            const int v = flag_wait(&a.hdr->order_ready, status);
            if (v == 0) {
                sm.abort = 1;
                if (blockIdx.x == 0)   // the status word says why; the scalars must not look like a result
                    for (int q = 0; q < 8; ++q) a.losses[q] = __int_as_float(0x7fc00000);
            }
            sm.n_tokens = max(v - 1, 0);
        } else {
            sm.n_tokens = a.hdr->n_tokens;
        }
    }
    __syncthreads();
    if (MODE == 1 && sm.abort) return;   // nothing is read or written through an order that is not this call's
    // number of work items of the streaming phase
    const int64_t n_items = MODE == 0 ? a.rows : (int64_t)sm.n_tokens;

    if (threadIdx.x >= kConsumers + 32) {
        // ------------------------------------------------------------ filler (step 6 only)
        if (MODE != 1) return;
        if (threadIdx.x == kConsumers + 32) {
        const LossArgs &la = a.loss;
        const int64_t n_masked = la.rows - n_items;
        const size_t row_bytes = (size_t)V * sizeof(T);
        const int64_t n_fill = filler_share(n_masked, a.fill_reserve_rows);
        for (;;) {
            const int64_t j = atomicAdd(&a.hdr->masked_next, 1);
            if (j >= n_fill) break;
            const int64_t row = a.order[la.rows - 1 - j];
            unsigned char *dst = reinterpret_cast<unsigned char *>(reinterpret_cast<T *>(la.dlogits) + row * (int64_t)V);
            for (size_t off = 0; off < row_bytes; off += kZeroBytes) {
                const uint32_t bytes = (uint32_t)min((size_t)kZeroBytes, row_bytes - off);
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst + off),
                             "r"(smem_addr(sm.zeros)), "r"(bytes)
                             : "memory");
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (la.dvalues) la.dvalues[row] = 0.f;
            if (la.new_logprob) la.new_logprob[row] = 0.f;
            if (la.entropy) la.entropy[row] = 0.f;
            if (la.dlogprob) la.dlogprob[row] = 0.f;
            float4 *p4 = reinterpret_cast<float4 *>(la.partials + row * kPartialsPerToken);
            p4[0] = make_float4(0.f, 0.f, 0.f, 0.f);
            p4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
            // keep a bounded number of row-sized groups in flight
            asm volatile("cp.async.bulk.wait_group.read 4;" ::: "memory");
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the block retires
        }
        __syncwarp();
        engine_epilogue<CONS>(a, sm);
        return;
    }

    if (threadIdx.x >= kConsumers) {
        // ------------------------------------------------------------ producer
        if (threadIdx.x == kConsumers) {
            const uint64_t policy = policy_evict_first();
            uint32_t k = 0;
            // Rows are handed out dynamically (SMs do not all stream at the same speed): step 6 draws
            // items from a counter in the workspace header, step 1 walks the rows with a grid stride
            // and settles rows with mask 0 on the way. -1 = nothing left.
            int64_t it_static = blockIdx.x;
            const auto fetch = [&]() -> int {
                if constexpr (MODE == 1) {
                    // the first two items of a block are fixed (no counter round trip before the first copy
                    // can be issued); everything after them is drawn from the counter
                    const int64_t item = 2 * (int64_t)gridDim.x + atomicAdd(&a.hdr->real_next, 1);
                    return item < n_items ? a.order[item] : -1;
                } else {
                    while (it_static < n_items) {
                        const int64_t row = it_static;
                        it_static += gridDim.x;
                        if (!a.mask || a.mask[row]) return (int)row;
                        a.logprob[row] = 0.f;
                        if (a.entropy) a.entropy[row] = 0.f;
                        if (a.lse) a.lse[row] = 0.f;
                    }
                    return -1;
                }
            };
            // the block's rows reach the consumers through sm.ring; the entry for item k + 1 is written
            // before the first copy of item k is armed, and read after that copy has landed
            int row_c, row_n;
            if (MODE == 1) {
                const int64_t i0 = blockIdx.x, i1 = i0 + gridDim.x;
                row_c = i0 < n_items ? a.order[i0] : -1;
                row_n = i1 < n_items ? a.order[i1] : -1;
            } else {
                row_c = fetch();
                row_n = row_c >= 0 ? fetch() : -1;
            }
            sm.ring[0] = row_c;
            if (row_c < 0) mbar_arrive(&sm.full[0]);   // no row at all: complete the phase the consumers wait for
            int64_t prev_row = -1;
            const auto load_chunk = [&](const unsigned char *src, int c) {
                const int packs = min(kChunkPacks, nvec - c * kChunkPacks);
                mbar_expect_tx(&sm.full[c], (uint32_t)packs * 16u);
                bulk_load(smem_raw + (size_t)c * kChunkBytes, src + (size_t)c * kChunkBytes, (uint32_t)packs * 16u,
                          &sm.full[c], policy);
            };
            // step 6: chunk c of the previous row now holds that row's gradient (written in place by
            // the consumers): ship it with one bulk shared->global copy
            const auto store_chunk = [&](int64_t row, int c) {
                const int packs = min(kChunkPacks, nvec - c * kChunkPacks);
                unsigned char *dst = reinterpret_cast<unsigned char *>(reinterpret_cast<T *>(a.loss.dlogits) + row * stride);
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst + (size_t)c * kChunkBytes),
                             "r"(smem_addr(smem_raw + (size_t)c * kChunkBytes)), "r"((uint32_t)packs * 16u)
                             : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            };
            while (row_c >= 0) {
                const int64_t row = row_c;
                sm.ring[(k + 1) & 3] = row_n;
                const int row_nn = row_n >= 0 ? fetch() : -1;   // needed one row from now
                const unsigned char *src = reinterpret_cast<const unsigned char *>(logits + row * stride);
                if (MODE == 0 || k == 0) {
                    for (int c = 0; c < nch; ++c) {
                        if (k > 0) mbar_wait(&sm.empty[c], (k - 1) & 1, status);
                        load_chunk(src, c);
                    }
                } else {
                    // the store of chunk c must have read shared memory before new bytes may land
                    // there: the load of a chunk trails its store by one chunk
                    for (int c = 0; c < nch; ++c) {
                        mbar_wait(&sm.empty[c], (k - 1) & 1, status);
                        store_chunk(prev_row, c);
                        if (c > 0) {
                            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                            load_chunk(src, c - 1);
                        }
                    }
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    load_chunk(src, nch - 1);
                }
                prev_row = row;
                row_c = row_n;
                row_n = row_nn;
                ++k;
            }
            if (MODE == 1 && k > 0) {   // gradient of the block's last row
                for (int c = 0; c < nch; ++c) {
                    mbar_wait(&sm.empty[c], (k - 1) & 1, status);
                    store_chunk(prev_row, c);
                }
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            }
            // The consumers have seen every chunk land, unless one of their waits ran out: make sure (bounded) that
            // no copy into this block's shared memory is still in flight when the block retires.
            if (k > 0)
                for (int c = 0; c < nch; ++c) mbar_wait(&sm.full[c], (k - 1) & 1, status);
        }
        if (MODE == 1) {
            __syncwarp();
            engine_epilogue<CONS>(a, sm);
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int ct = threadIdx.x;
    const uint4 *buf = reinterpret_cast<const uint4 *>(smem_raw);
    const T *buf_elems = reinterpret_cast<const T *>(smem_raw);
    const double inv_n = MODE == 1 ? 1.0 / (double)sm.n_tokens : 0.0;
    const float inv_n_f = (float)inv_n;
    uint32_t k = 0;
    // The block's rows come from sm.ring (see the producer). Per-row scalars are dependent loads
    // (row -> token id, old log-prob, ...): they are requested for the NEXT row as soon as its index is
    // known (first chunk of the current row) and become current at the end of the iteration.
    int row_c, row_n = -1;
    int tok_c = -1, tok_n = -1;
    float in_c[5] = {0.f, 0.f, 0.f, 0.f, 0.f}, in_n[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
    // advantages and returns of this step: polled while the first row's bytes are on their way
    if (MODE == 1 && a.wait_flags && ct == 0) flag_wait(&a.hdr->adv_ready, status);
    mbar_wait(&sm.full[0], 0, status);
    if (MODE == 1) consumer_sync<CONS>();
    row_c = sm.ring[0];
    if (row_c >= 0) {
        tok_c = a.tokens[row_c];
        if (MODE == 1) {
            if (a.loss.g_ext) {
                in_c[0] = a.loss.g_ext[row_c];
            } else {
                in_c[0] = a.loss.old_logprob[row_c];
                in_c[1] = a.loss.advantages[row_c];
            }
        }
        if (MODE == 1 && ct == 0 && !a.loss.g_ext) {
            in_c[2] = a.loss.values_new[row_c];
            in_c[3] = a.loss.values_old[row_c];
            in_c[4] = a.loss.returns[row_c];
        }
    }
    while (row_c >= 0) {
        const int64_t row = row_c;
        const int tok = tok_c;
        const float t_old = in_c[0], t_adv = in_c[1], t_vn = in_c[2], t_vo = in_c[3], t_ret = in_c[4];
        const bool bad = tok < 0 || tok >= V;
        const int tok_chunk = bad ? -1 : (tok / N) / kChunkPacks;
        float xtok = 0.f;
        // ---- pass 1: statistics, chunk by chunk as the bytes land
        ThreadStats<T, ENTROPY> ts;
        const uint32_t parity = k & 1;
        float m_common = 0.f;
        for (int c = 0; c < nch; ++c) {
            mbar_wait(&sm.full[c], parity, status);
            if (c == 0) {   // every thread reads the row's first pack: one reference for the whole row
                float x[N], xmax;
                Pack<T>::unpack(buf[0], x, xmax);
                m_common = safe_reference(xmax, a.c);
                ts.init(m_common);
                // the next row is known now: request its scalars
                row_n = sm.ring[(k + 1) & 3];
                if (row_n >= 0) {
                    tok_n = a.tokens[row_n];
                    if (MODE == 1) {   // every thread derives the gradient scale itself, so every thread needs these two
                        if (a.loss.g_ext) {
                            in_n[0] = a.loss.g_ext[row_n];
                        } else {
                            in_n[0] = a.loss.old_logprob[row_n];
                            in_n[1] = a.loss.advantages[row_n];
                        }
                    }
                    if (MODE == 1 && ct == 0 && !a.loss.g_ext) {
                        in_n[2] = a.loss.values_new[row_n];
                        in_n[3] = a.loss.values_old[row_n];
                        in_n[4] = a.loss.returns[row_n];
                    }
                }
            }
            const int i0 = c * kChunkPacks + ct, i1 = i0 + kConsumers;
            const bool h0 = i0 < nvec, h1 = i1 < nvec;
            uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
            if (h0) v0 = buf[i0];
            if (h1) v1 = buf[i1];
            if ((MODE == 1 || ct == 0) && c == tok_chunk) xtok = Pack<T>::load1(buf_elems + tok);
            ts.chunk(v0, h0, v1, h1, a.c);
            if (MODE == 0) {
                __syncwarp();
                if ((ct & 31) == 0) mbar_arrive(&sm.empty[c]);
            }
        }
        const SoftmaxState st = consumer_merge_common<MODE == 1, CONS>(ts.state(), m_common, sm.red[parity], ct);
        const float l2s = log2f(st.s);
        if (MODE == 0) {
            if (ct == 0) {
                float lp = (fmaf(xtok, a.c, -st.m) - l2s) * kLn2;
                float H = (l2s - st.u / st.s) * kLn2;
                float L = (st.m + l2s) * kLn2;
                if (bad) {
                    lp = H = L = __int_as_float(0x7fc00000);
                    if (status) atomicOr(status, PPO_DEV_BAD_TOKEN);
                }
                a.logprob[row] = lp;
                if (a.entropy) a.entropy[row] = H;
                if (a.lse) a.lse[row] = L;
            }
        } else {
            const LossArgs &la = a.loss;
            // Every consumer thread derives the gradient scale from the row sums by itself (a few dozen
            // fp32 instructions, identical in all threads): no second barrier and no single-thread
            // section between the two passes over the row.
            float lp = (fmaf(xtok, a.c, -st.m) - l2s) * kLn2;
            if (bad) lp = __int_as_float(0x7fc00000);
            PolicyTerm pt;
            if (la.g_ext) {   // the gradient on the log-prob is an input (a bad token still poisons its row)
                pt.g = bad ? lp : t_old;
                pt.pg = pt.kl = pt.pg_clipped = 0.f;
            } else {
                pt = policy_term(lp, t_old, t_adv, la.eps, inv_n_f);
            }
            const float Y = st.m + l2s;           // log2-sum-exp
            const float gs = pt.g * la.inv_tau;   // gradient scale
            if (ct == 0) {   // per-token outputs; the other warps are already in pass 2
                float H = (l2s - st.u / st.s) * kLn2;
                if (bad) {
                    H = lp;
                    if (status) atomicOr(status, PPO_DEV_BAD_TOKEN);
                }
                ValueTerm vt;
                vt.dvalue = vt.vf = vt.vf_clipped = 0.f;
                if (!la.g_ext) vt = value_term(t_vn, t_vo, t_ret, la.eps_v, la.c1, inv_n);
                if (la.dvalues) la.dvalues[row] = vt.dvalue;
                if (la.new_logprob) la.new_logprob[row] = lp;
                if (la.entropy) la.entropy[row] = H;
                if (la.dlogprob) la.dlogprob[row] = pt.g;
                float4 *p4 = reinterpret_cast<float4 *>(la.partials + row * kPartialsPerToken);
                p4[0] = make_float4(pt.pg, vt.vf, pt.kl, pt.pg_clipped);
                p4[1] = make_float4(vt.vf_clipped, H, 0.f, 0.f);
            }
            // ---- pass 2: gradient row, chunk by chunk; each chunk is handed back to the producer
            // the gradient is written over the logits in shared memory; the producer ships each chunk
            T *dst = reinterpret_cast<T *>(smem_raw);
            uint4 *dst4 = reinterpret_cast<uint4 *>(smem_raw);
            // -gs * 2^(y - Y) = -+ 2^(y - Y + log2|gs|): the scale rides in the exponent
            const float off = log2f(fabsf(gs)) - Y;
            const bool zero = gs == 0.f, neg = gs > 0.f;
            const bool fix_owner = !zero && !bad && ct == (tok / N) % kConsumers;
            for (int c = 0; c < nch; ++c) {
                const int i0 = c * kChunkPacks + ct;
                float xt_fix = 0.f;   // the token's logit, read before its pack is overwritten in place
                if (fix_owner && c == tok_chunk) xt_fix = Pack<T>::load1(buf_elems + tok);
                // three uniform variants of the same loop: the sign of the scale and the all-zero row
                // (clipped token, g = 0) are decided once per row, not per element
                if (zero) {
                    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                    if (i0 < nvec) dst4[i0] = z;
                    if (i0 + kConsumers < nvec) dst4[i0 + kConsumers] = z;
                } else if (neg) {
                    gradient_packs<T, true, CONS>(buf, dst4, i0, nvec, a.c, off);
                } else {
                    gradient_packs<T, false, CONS>(buf, dst4, i0, nvec, a.c, off);
                }
                // the thread that wrote the pack holding the sampled token adds the one-hot term
                if (fix_owner && c == tok_chunk) {
                    const float e = ex2(fmaf(xt_fix, a.c, off));
                    Pack<T>::store1(dst + tok, gs + (neg ? -e : e));
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the bulk store
                __syncwarp();
                if ((ct & 31) == 0) mbar_arrive(&sm.empty[c]);
            }
        }
        row_c = row_n;
        tok_c = tok_n;
#pragma unroll
        for (int q = 0; q < 5; ++q) in_c[q] = in_n[q];
        ++k;
    }

    if (MODE == 1) {
        // ---- zero-fill phase: rows with mask 0, handed out by a shared counter
        const LossArgs &la = a.loss;
        const int64_t n_masked = a.loss.rows - n_items;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
        // masked item j is row order[rows - 1 - j]: the fillers draw j in [0, n_fill) from masked_next, the rows kept
        // back are j in [n_fill, n_masked) and are drawn from masked_tail; once those are gone the consumers help
        // with whatever the fillers have left
        const int64_t n_fill = filler_share(n_masked, a.fill_reserve_rows);
        bool tail = n_fill < n_masked;
        for (;;) {
            consumer_sync<CONS>();
            if (ct == 0)
                sm.next_item = tail ? (int)n_fill + atomicAdd(&a.hdr->masked_tail, 1) : atomicAdd(&a.hdr->masked_next, 1);
            consumer_sync<CONS>();
            const int64_t j = sm.next_item;
            if (tail) {
                if (j >= n_masked) {
                    tail = false;
                    continue;
                }
            } else if (j >= n_fill)
                break;
            const int64_t row = a.order[a.loss.rows - 1 - j];
            uint4 *dst4 = reinterpret_cast<uint4 *>(reinterpret_cast<T *>(la.dlogits) + row * (int64_t)V);
            for (int i = ct; i < nvec; i += kConsumers) st_stream(dst4 + i, z);
            if (ct == 0) {
                if (la.dvalues) la.dvalues[row] = 0.f;
                if (la.new_logprob) la.new_logprob[row] = 0.f;
                if (la.entropy) la.entropy[row] = 0.f;
                if (la.dlogprob) la.dlogprob[row] = 0.f;
                float4 *p4 = reinterpret_cast<float4 *>(la.partials + row * kPartialsPerToken);
                p4[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                p4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        engine_epilogue<CONS>(a, sm);
    }
}

// ---------------------------------------------------------------- host side
static int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

template <typename T, int MODE, bool ENTROPY>
static int launch_engine(const EngineArgs &a, int64_t max_items, bool dependent, cudaStream_t s)
{
    const size_t row_bytes = (size_t)a.V * sizeof(T);
    if (row_bytes > kMaxRowBytes) return PPO_ERR_UNSUPPORTED;
    const size_t smem = (row_bytes + 127) & ~size_t(127);   // the last chunk may be partial
    const bool two = smem <= 110 * 1024;
    int64_t grid = (int64_t)sm_count() * (two ? 2 : 1);
    if (MODE == 0 && max_items < grid) grid = max_items;
    if (grid < 1) grid = 1;
    if (two) {
        // two blocks per SM: 16 consumer warps each, 16 KB chunks
        auto kern = row_engine_kernel<T, MODE, ENTROPY, 2, 512>;
        PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dependent) PPO_RETURN_IF_CUDA(launch_dependent(kern, dim3((unsigned)grid), dim3(512 + 64), smem, s, a));
        else kern<<<(unsigned)grid, 512 + 64, smem, s>>>(a);
    } else {
        // one block per SM: 30 consumer warps (a block holds at most 1024 threads), 30 KB chunks
        auto kern = row_engine_kernel<T, MODE, ENTROPY, 1, 960>;
        PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dependent) PPO_RETURN_IF_CUDA(launch_dependent(kern, dim3((unsigned)grid), dim3(960 + 64), smem, s, a));
        else kern<<<(unsigned)grid, 960 + 64, smem, s>>>(a);
    }
    return launch_status();
}

template <typename T>
static bool bulk_ok(const void *base, int64_t stride_elems, int V)
{
    return aligned16(base) && (stride_elems * (int64_t)sizeof(T)) % 16 == 0 && V % Pack<T>::N == 0 &&
           (size_t)V * sizeof(T) <= kMaxRowBytes;
}

int launch_logprob_bulk(const void *logits, int dtype, int64_t rows, int V, int64_t row_stride,
                        const int32_t *tokens, const uint8_t *mask, float c, float *logprob, float *entropy,
                        float *lse, int *status, cudaStream_t s)
{
    EngineArgs a = {};
    a.logits = logits;
    a.rows = rows;
    a.row_stride = row_stride;
    a.V = V;
    a.tokens = tokens;
    a.mask = mask;
    a.c = c;
    a.logprob = logprob;
    a.entropy = entropy;
    a.lse = lse;
    a.status = status;
    if (dtype == PPO_F32) {
        if (!bulk_ok<float>(logits, row_stride, V)) return PPO_ERR_UNSUPPORTED;
        return entropy ? launch_engine<float, 0, true>(a, rows, false, s) : launch_engine<float, 0, false>(a, rows, false, s);
    }
    if (!bulk_ok<__nv_bfloat16>(logits, row_stride, V)) return PPO_ERR_UNSUPPORTED;
    return entropy ? launch_engine<__nv_bfloat16, 0, true>(a, rows, false, s)
                   : launch_engine<__nv_bfloat16, 0, false>(a, rows, false, s);
}

int launch_loss_bulk(const LossArgs &la, int dtype, void *workspace, float *losses, float vf_coef, bool dependent,
                     cudaStream_t s, bool reuse, bool keep_back)
{
    if (!la.dlogits || !aligned16(la.dlogits)) return PPO_ERR_UNSUPPORTED;
    EngineArgs a = {};
    a.logits = la.logits;
    a.rows = la.rows;
    a.row_stride = la.V;
    a.V = la.V;
    a.tokens = la.tokens;
    a.mask = la.mask;
    a.c = la.c;
    a.status = la.status;
    a.loss = la;
    a.order = ws_order(workspace, la.rows);
    a.hdr = ws_header(workspace);
    a.losses = losses;
    a.vf_coef = vf_coef;
    a.wait_flags = dependent ? 1 : 0;
    a.reuse = reuse ? 1 : 0;
    a.fill_reserve_rows = keep_back ? kReuseReserveRows : 0;
    if (dtype == PPO_F32) {
        if (!bulk_ok<float>(la.logits, la.V, la.V)) return PPO_ERR_UNSUPPORTED;
        return launch_engine<float, 1, true>(a, la.rows, dependent, s);
    }
    if (!bulk_ok<__nv_bfloat16>(la.logits, la.V, la.V)) return PPO_ERR_UNSUPPORTED;
    return launch_engine<__nv_bfloat16, 1, true>(a, la.rows, dependent, s);
}

}   // namespace ppo
