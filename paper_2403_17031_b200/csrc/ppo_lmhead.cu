// Step 7: LM-head GEMM fused with the log-prob / entropy reduction. The logits H.W are formed tile
// by tile on the 5th-generation tensor cores and consumed straight out of tensor memory; they are
// never written to global memory.
//
// One persistent block per SM, 192 threads (320 when a work unit covers two row tiles, see LmShape) in three roles:
//   warp 0 (one lane)   TMA producer: 128x64 tiles of H (K-major) and 64x256 tiles of W (vocabulary-
//                       major, as stored: W is [K,V] row-major) into a 4-stage shared-memory ring,
//                       128-byte swizzle, completion counted on mbarriers
//   warp 1 (one lane)   issues tcgen05.mma (M=128, N=256, K=16, bf16 x bf16 -> fp32) into one of two
//                       256-column accumulators in tensor memory; tcgen05.commit releases the ring
//                       slot and, after the last k-block, hands the accumulator to the epilogue
//   warps 2-5           epilogue: thread r owns logits row r of the tile; tcgen05.ld 32 columns at a
//                       time and fold them into that row's running softmax state (fixed reference,
//                       one ex2 per logit), picking up the sampled token's logit on the way
// While the epilogue drains one accumulator the tensor core fills the other.
//
// Work unit = (row tile of 128, chunk of 6 vocabulary tiles of 256). Units are ordered so that the
// blocks running at the same time share the same W columns and a small set of H tiles (both stay
// in L2); block b takes units b, b+grid, ... Each unit leaves one partial state per row in the
// workspace; a second small kernel merges a row's partials in chunk order and writes log-prob,
// entropy and lse.
//
// Given a mask, the call first packs the rows with mask 1 into the workspace (row order and count found on the
// device) and this kernel multiplies only those; it reads the row count from the workspace header, so its unit
// list is as long as the packed rows need, and the second kernel writes each result at its original row.
//
// Every wait is bounded; a wait that runs out sets PPO_DEV_TIMEOUT and the block carries on with the
// same control flow, so it still reaches the end, frees its tensor memory and returns.
#include "ppo_tcgen05.cuh"

namespace ppo {

constexpr int kBlockM = 128, kBlockN = 256, kBlockK = 64;
constexpr int kMaxStages = 4;
constexpr int kABytes = kBlockM * kBlockK * 2;          // 16 KB
constexpr int kBBoxBytes = 64 * kBlockK * 2;            // 8 KB: one 64(N) x 64(K) box of W
constexpr int kBBytes = (kBlockN / 64) * kBBoxBytes;    // 32 KB
// MT = row tiles of 128 that one work unit multiplies with the same W tile. MT = 2 (the default for
// M > 128): two accumulators of 256 columns fill the tensor memory, every W tile staged in shared memory
// feeds two MMAs, and the ring moves 64 KB instead of 96 KB per 2 x (128 x 256 x 64) multiply-adds - the
// ring, not the tensor pipe, is what limits this kernel. The price: no second accumulator set, so the
// epilogue (eight warps, four per accumulator) is not hidden behind the next tile's MMAs.
template <int MT> struct LmShape {
    static constexpr int kStages = MT == 1 ? 4 : 3;
    static constexpr int kStageBytes = MT * kABytes + kBBytes;      // 48 KB / 64 KB
    static constexpr int kThreads = 64 + MT * 128;                  // TMA warp, MMA warp, 4 * MT epilogue warps
    static constexpr int kSets = MT == 1 ? 2 : 1;                   // accumulator sets in the 512 columns
};
constexpr int kTilesPerChunk = 6;                       // vocabulary tiles per work unit
constexpr int kRowGroup = 37;                           // row tiles that sweep the vocabulary together
constexpr uint32_t kAbsentBits = 0xffffffffu;           // "this chunk does not hold the sampled token"

struct LmSmem {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
};

// instruction descriptor: D fp32, A and B bf16, A K-major, B MN-major, M = 128, N = 256
constexpr uint32_t kInstrDesc = tc::instr_desc(false, true, kBlockM, kBlockN);

struct LmUnit {
    int m_tile, chunk;
};

// unit index -> (row tile, vocabulary chunk): row tiles in groups of kRowGroup; inside a group the
// chunk index moves slowest, so consecutive units share W columns
__device__ __forceinline__ LmUnit lm_unit(int u, int m_tiles, int n_chunks)
{
    const int per_group = kRowGroup * n_chunks;
    const int g = u / per_group;
    const int gsize = min(kRowGroup, m_tiles - g * kRowGroup);
    const int local = u - g * per_group;
    LmUnit r;
    r.chunk = local / gsize;
    r.m_tile = g * kRowGroup + (local - r.chunk * gsize);
    return r;
}

struct LmArgs {
    int M, K, V;
    int m_tiles, n_tiles, n_chunks, n_units;
    // Row compaction (the call was given a mask): H holds the rows with mask 1 only, packed by an earlier kernel of
    // the stream; *m_eff = how many (known on the device only: M, m_tiles and n_units above are upper bounds),
    // order[j] = the original index of packed row j (tokens is indexed by the original row)
    const int *m_eff;
    const int32_t *order;
    const int32_t *tokens;
    float c;
    float4 *partials;     // [m_tiles*128][n_chunks]
    int *status;
};

template <int MT>
__global__ void __launch_bounds__(LmShape<MT>::kThreads, 1)
lmhead_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, const LmArgs a)
{
    constexpr int kStages = LmShape<MT>::kStages, kStageBytes = LmShape<MT>::kStageBytes, kSets = LmShape<MT>::kSets;
    extern __shared__ __align__(1024) unsigned char lm_smem_raw[];
    __shared__ LmSmem sm;
    // the ring must start on a 1024-byte boundary (swizzle atoms)
    unsigned char *ring = lm_smem_raw + ((1024u - (tc::saddr(lm_smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_blocks = a.K / kBlockK;
    // every role walks the same unit list, derived from the same row count
    int n_rows = a.M, m_tiles = a.m_tiles, n_units = a.n_units;
    if (a.m_eff) {
        n_rows = max(0, min(*a.m_eff, a.M));
        m_tiles = ((n_rows + kBlockM - 1) / kBlockM + MT - 1) / MT;
        n_units = m_tiles * a.n_chunks;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            tc::barrier_init(&sm.full[s], 1);
            tc::barrier_init(&sm.empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            tc::barrier_init(&sm.tmem_full[b], 1);
            tc::barrier_init(&sm.tmem_empty[b], 4 * MT);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // one warp allocates all 512 columns of tensor memory
        tc::tmem_alloc_all(&sm.tmem_base);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                const LmUnit un = lm_unit(u, m_tiles, a.n_chunks);
                const int t0 = un.chunk * kTilesPerChunk, t1 = min(t0 + kTilesPerChunk, a.n_tiles);
                for (int t = t0; t < t1; ++t) {
                    for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                        const int s = it % kStages;
                        if (it >= kStages) tc::wait(&sm.empty[s], ((it / kStages) - 1) & 1, a.status);
                        unsigned char *stage = ring + (size_t)s * kStageBytes;
                        tc::barrier_expect_tx(&sm.full[s], (uint32_t)kStageBytes);
#pragma unroll
                        for (int j = 0; j < MT; ++j)   // (a tile past the last row is filled with zeros)
                            tc::tma_load_2d(stage + j * kABytes, &map_h, kb * kBlockK, (un.m_tile * MT + j) * kBlockM,
                                        &sm.full[s]);
#pragma unroll
                        for (int j = 0; j < kBlockN / 64; ++j)
                            tc::tma_load_2d(stage + MT * kABytes + j * kBBoxBytes, &map_w, t * kBlockN + j * 64,
                                        kb * kBlockK, &sm.full[s]);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tc = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                const LmUnit un = lm_unit(u, m_tiles, a.n_chunks);
                const int t0 = un.chunk * kTilesPerChunk, t1 = min(t0 + kTilesPerChunk, a.n_tiles);
                for (int t = t0; t < t1; ++t, ++tc) {
                    const uint32_t buf = tc % kSets;
                    if (tc >= (uint32_t)kSets) tc::wait(&sm.tmem_empty[buf], ((tc / kSets) - 1) & 1, a.status);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t tmem_d = tmem_base + buf * (MT * kBlockN);
                    for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                        const int s = it % kStages;
                        tc::wait(&sm.full[s], (it / kStages) & 1, a.status);
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a_addr = tc::saddr(ring + (size_t)s * kStageBytes);
                        const uint32_t b_addr = a_addr + MT * kABytes;
#pragma unroll
                        for (int kk = 0; kk < kBlockK / 16; ++kk) {
                            // B: vocabulary-major; 64-column boxes 8192 B apart, 8 K-rows 1024 B apart;
                            //    16 K-rows = 2048 bytes further
                            const uint64_t bd = tc::smem_desc(b_addr + kk * 2048, kBBoxBytes, 1024);
#pragma unroll
                            for (int j = 0; j < MT; ++j) {
                                // A: K-major, 8-row groups 1024 B apart; 16 K-elements = 32 bytes further
                                const uint64_t ad = tc::smem_desc(a_addr + j * kABytes + kk * 32, 16, 1024);
                                tc::mma(tmem_d + j * kBlockN, ad, bd, kInstrDesc, (kb | kk) ? 1u : 0u);
                            }
                        }
                        tc::commit(&sm.empty[s]);            // ring slot is free once these MMAs have read it
                    }
                    tc::commit(&sm.tmem_full[buf]);          // accumulator complete
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                      // tensor-memory lane quarter this warp may read
        const int acc = (warp - 2) >> 2;             // which of the unit's MT accumulators / row tiles
        const int row_in_tile = q * 32 + lane;
        uint32_t tc = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const LmUnit un = lm_unit(u, m_tiles, a.n_chunks);
            const int t0 = un.chunk * kTilesPerChunk, t1 = min(t0 + kTilesPerChunk, a.n_tiles);
            const int row = (un.m_tile * MT + acc) * kBlockM + row_in_tile;
            const bool row_ok = row < n_rows;
            const int tok = row_ok ? a.tokens[a.order ? a.order[row] : row] : -1;
            float m = 0.f, s0 = 0.f, s1 = 0.f, u0 = 0.f, u1 = 0.f;
            bool have_ref = false;
            uint32_t xtok_bits = kAbsentBits;
            for (int t = t0; t < t1; ++t, ++tc) {
                const uint32_t buf = tc % kSets;
                tc::wait(&sm.tmem_full[buf], (tc / kSets) & 1, a.status);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t taddr = tmem_base + buf * (MT * kBlockN) + acc * kBlockN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
                for (int cc = 0; cc < kBlockN / 32; ++cc) {
                    uint32_t r[32];
                    __syncwarp();                            // the aligned tensor-memory load needs a converged warp
                    tc::tmem_ld32(taddr + cc * 32, r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (cc == kBlockN / 32 - 1) {
                        // all of this warp's reads of the accumulator are done: hand it back
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) tc::barrier_arrive(&sm.tmem_empty[buf]);
                    }
                    const int col0 = t * kBlockN + cc * 32;
                    if (col0 >= a.V) continue;
                    const int ncol = min(32, a.V - col0);
                    if ((unsigned)(tok - col0) < (unsigned)ncol) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (tok - col0 == j) xtok_bits = r[j];
                    }
                    if (!have_ref) {
                        float mx = __uint_as_float(r[0]);
#pragma unroll
                        for (int j = 1; j < 32; ++j)
                            if (j < ncol) mx = fmaxf(mx, __uint_as_float(r[j]));
                        m = mx * a.c;
                        have_ref = true;
                    }
                    for (int attempt = 0; attempt < 2; ++attempt) {
                        const float nm = -m;
                        float a0 = s0, a1 = s1, b0 = u0, b1 = u1;
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const float ta = fmaf(__uint_as_float(r[j]), a.c, nm);
                            const float tb = fmaf(__uint_as_float(r[j + 1]), a.c, nm);
                            const float ea = j < ncol ? ex2(ta) : 0.f, eb = j + 1 < ncol ? ex2(tb) : 0.f;
                            a0 += ea;
                            a1 += eb;
                            b0 = fmaf(ea, j < ncol ? ta : 0.f, b0);
                            b1 = fmaf(eb, j + 1 < ncol ? tb : 0.f, b1);
                        }
                        if (a0 + a1 < 1.0e35f || attempt == 1) {
                            s0 = a0; s1 = a1; u0 = b0; u1 = b1;
                            break;
                        }
                        // overflow: move the reference up to this chunk's maximum and redo the chunk
                        float mx = __uint_as_float(r[0]);
#pragma unroll
                        for (int j = 1; j < 32; ++j)
                            if (j < ncol) mx = fmaxf(mx, __uint_as_float(r[j]));
                        const float m2 = fmaxf(m, mx * a.c);
                        const float d = m - m2, sc = ex2(d);
                        u0 = sc * fmaf(d, s0, u0);
                        u1 = sc * fmaf(d, s1, u1);
                        s0 *= sc;
                        s1 *= sc;
                        m = m2;
                    }
                }
            }
            if (row_ok)
                a.partials[(size_t)row * a.n_chunks + un.chunk] =
                    make_float4(m, s0 + s1, u0 + u1, __uint_as_float(xtok_bits));
        }
    }

    // ---------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tc::tmem_free_all(tmem_base);
    }
}

// pack the rows with mask 1 (order[0 .. *n)) of H [M, K] into Hc, zeros up to the next multiple of 128 rows;
// k16 = 16-byte pieces per row
__global__ void __launch_bounds__(256)
lmhead_pack_rows_kernel(const uint4 *__restrict__ H, int k16, const int32_t *__restrict__ order, const int *__restrict__ n,
                        uint4 *__restrict__ Hc)
{
    const int j = blockIdx.x, rows = *n;
    uint4 *dst = Hc + (size_t)j * k16;
    if (j < rows) {
        const uint4 *src = H + (size_t)order[j] * k16;
        for (int i = threadIdx.x; i < k16; i += blockDim.x) dst[i] = src[i];
    } else if (j < ((rows + kBlockM - 1) / kBlockM) * kBlockM) {
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
        for (int i = threadIdx.x; i < k16; i += blockDim.x) dst[i] = z;
    }
}

// merge the chunk partials of each row in chunk order; one thread per row. With row compaction thread i holds
// packed row i < *m_eff (original row order[i]); the threads beyond write the zeros of the rows with mask 0.
__global__ void __launch_bounds__(256)
lmhead_finalize_kernel(const float4 *__restrict__ partials, int M, int V, int n_chunks, const int32_t *__restrict__ tokens,
                       const uint8_t *__restrict__ mask, const int32_t *__restrict__ order,
                       const int *__restrict__ m_eff, float c, float *__restrict__ logprob,
                       float *__restrict__ entropy, float *__restrict__ lse, int *status,
                       unsigned long long *order_sig)
{
    // the partials of this call lie where a loss call keeps its row order: that order is void from here on
    if (blockIdx.x == 0 && threadIdx.x == 0) order_sig[0] = 0ull;
    const int packed = blockIdx.x * blockDim.x + threadIdx.x;
    if (packed >= M) return;
    const int row = order ? order[packed] : packed;
    const bool real = order ? packed < *m_eff : (!mask || mask[row]);
    float lp = 0.f, H = 0.f, L = 0.f;
    if (real) {
        SoftmaxState st;
        st.init();
        uint32_t xbits = kAbsentBits;
        for (int k = 0; k < n_chunks; ++k) {
            const float4 p = partials[(size_t)packed * n_chunks + k];
            SoftmaxState o;
            o.m = p.x;
            o.s = p.y;
            o.u = p.z;
            st = merge(st, o);
            if (__float_as_uint(p.w) != kAbsentBits) xbits = __float_as_uint(p.w);
        }
        const int tok = tokens[row];
        const float l2s = log2f(st.s);
        if (tok < 0 || tok >= V || xbits == kAbsentBits) {
            lp = H = L = __int_as_float(0x7fc00000);
            atomicOr(status, PPO_DEV_BAD_TOKEN);
        } else {
            lp = (fmaf(__uint_as_float(xbits), c, -st.m) - l2s) * kLn2;
            H = (l2s - st.u / st.s) * kLn2;
            L = (st.m + l2s) * kLn2;
        }
    }
    logprob[row] = lp;
    if (entropy) entropy[row] = H;
    if (lse) lse[row] = L;
}

// ---------------------------------------------------------------- host side
using tc::make_map;

static size_t lm_partials_bytes(int m_tiles, int n_chunks)
{
    return align256((size_t)m_tiles * kBlockM * (size_t)n_chunks * sizeof(float4));
}

static void lm_shape(int64_t M, int64_t V, int *m_tiles, int *n_tiles, int *n_chunks)
{
    *m_tiles = (int)((M + kBlockM - 1) / kBlockM);
    *n_tiles = (int)((V + kBlockN - 1) / kBlockN);
    *n_chunks = (*n_tiles + kTilesPerChunk - 1) / kTilesPerChunk;
}

LmWorkspace lm_workspace(int64_t M, int64_t K, int64_t V)
{
    int m_tiles, n_tiles, n_chunks;
    lm_shape(M, V, &m_tiles, &n_tiles, &n_chunks);
    LmWorkspace w;
    w.order_off = kHeaderBytes + lm_partials_bytes(m_tiles, n_chunks);
    w.packed_off = w.order_off + align256((size_t)M * sizeof(int32_t));
    w.bytes = w.packed_off + align256((size_t)M * (size_t)(K > 0 ? K : 0) * 2);
    return w;
}

int launch_lm_pack_rows(const void *H, int64_t M, int64_t K, const uint8_t *mask, void *workspace,
                        const LmWorkspace &lay, cudaStream_t s)
{
    unsigned char *ws = reinterpret_cast<unsigned char *>(workspace);
    int32_t *order = reinterpret_cast<int32_t *>(ws + lay.order_off);
    int rc = launch_row_order(mask, M, ws_header(workspace), order, s);
    if (rc) return rc;
    lmhead_pack_rows_kernel<<<(unsigned)M, 256, 0, s>>>(reinterpret_cast<const uint4 *>(H), (int)(K / 8), order,
                                                      &ws_header(workspace)->n_tokens,
                                                      reinterpret_cast<uint4 *>(ws + lay.packed_off));
    return launch_status();
}

}   // namespace ppo

using namespace ppo;

extern "C" size_t ppo_lmhead_workspace_bytes(int64_t M, int64_t K, int64_t V)
{
    if (M <= 0 || V <= 0) return kHeaderBytes;
    return lm_workspace(M, K, V).bytes;
}

extern "C" int ppo_lmhead_logprob_entropy(const void *H, const void *W, int64_t M, int64_t K, int64_t V,
                                          const int32_t *tokens, const uint8_t *mask, float temperature,
                                          float *logprob, float *entropy, float *lse, void *workspace,
                                          void *stream)
{
    if (M < 0 || K <= 0 || V <= 0 || M >= ((int64_t)1 << 31) - kBlockM || V >= ((int64_t)1 << 31) - kBlockN ||
        K >= ((int64_t)1 << 31))
        return PPO_ERR_SHAPE;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    if (M == 0) return PPO_OK;
    if (!H || !W || !tokens || !logprob || !workspace) return PPO_ERR_NULL;
    if (K % kBlockK != 0 || V % 8 != 0) return PPO_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(H) % 16 || reinterpret_cast<uintptr_t>(W) % 16 ||
        reinterpret_cast<uintptr_t>(workspace) % 256)
        return PPO_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    LmArgs a;
    a.M = (int)M;
    a.K = (int)K;
    a.V = (int)V;
    lm_shape(M, V, &a.m_tiles, &a.n_tiles, &a.n_chunks);
    const int64_t units = (int64_t)a.m_tiles * a.n_chunks;
    if (units >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    a.n_units = (int)units;
    a.tokens = tokens;
    a.c = kLog2e / temperature;
    unsigned char *ws = reinterpret_cast<unsigned char *>(workspace);
    a.partials = reinterpret_cast<float4 *>(ws + kHeaderBytes);
    a.status = &ws_header(workspace)->status;
    a.m_eff = nullptr;
    a.order = nullptr;
    int rc;
    // With a mask, and more than one row tile, the rows with mask 0 are taken out of the GEMM: their order is
    // found on the device, the other rows of H are packed into the workspace (M*K*2 bytes moved against
    // 2*K*V flops saved per row with mask 0) and the kernels below work on the packed rows; the finalize kernel
    // writes every result at its original row.
    if (mask && a.m_tiles >= 2) {
        const LmWorkspace lay = lm_workspace(M, K, V);
        rc = launch_lm_pack_rows(H, M, K, mask, workspace, lay, s);
        if (rc) return rc;
        a.m_eff = &ws_header(workspace)->n_tokens;
        a.order = reinterpret_cast<const int32_t *>(ws + lay.order_off);
        H = ws + lay.packed_off;
    }

    CUtensorMap map_h, map_w;
    rc = make_map(&map_h, H, (uint64_t)K, (uint64_t)M, kBlockM);
    if (rc) return rc;
    rc = make_map(&map_w, W, (uint64_t)V, (uint64_t)K, kBlockK);
    if (rc) return rc;

    int dev = 0, sms = 148;
    PPO_RETURN_IF_CUDA(cudaGetDevice(&dev));
    PPO_RETURN_IF_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // two row tiles per unit pay off when the units still spread evenly over the SMs (a unit is twice as long)
    if (a.m_tiles >= 2 && (int64_t)((a.m_tiles + 1) / 2) * a.n_chunks >= 12 * (int64_t)sms) {
        // the unit grid is over pairs of row tiles
        a.m_tiles = (a.m_tiles + 1) / 2;
        a.n_units = a.m_tiles * a.n_chunks;
        const size_t smem = (size_t)LmShape<2>::kStages * LmShape<2>::kStageBytes + 1024;   // + slack to align the ring
        PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(lmhead_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        const int grid = a.n_units < sms ? a.n_units : sms;
        lmhead_kernel<2><<<grid, LmShape<2>::kThreads, smem, s>>>(map_h, map_w, a);
    } else {
        const size_t smem = (size_t)LmShape<1>::kStages * LmShape<1>::kStageBytes + 1024;
        PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(lmhead_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        const int grid = a.n_units < sms ? a.n_units : sms;
        lmhead_kernel<1><<<grid, LmShape<1>::kThreads, smem, s>>>(map_h, map_w, a);
    }
    rc = launch_status();
    if (rc) return rc;
    lmhead_finalize_kernel<<<(unsigned)((M + 255) / 256), 256, 0, s>>>(a.partials, a.M, a.V, a.n_chunks, tokens, mask, a.order,
                                                                       a.m_eff, a.c, logprob, entropy, lse, a.status,
                                                                       ws_header(workspace)->order_sig);
    return launch_status();
}
