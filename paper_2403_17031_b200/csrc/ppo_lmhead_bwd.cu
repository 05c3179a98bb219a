// Backward of the fused LM head (the step after the loss at log-prob level, for config 4): given the
// gradient g on each token's log-prob,
//     D  = g * (onehot(token) - softmax(H W / tau)) / tau        [M, V]   (gradient on the logits)
//     dH = D W^T                                                 [M, K]
//     dW = H^T D                                                 [K, V]
// as three launches of one tcgen05 GEMM kernel:
//   pass 1  recomputes the logits tile by tile (H W, as in the forward kernel) and turns each
//           accumulator tile into its tile of D in the epilogue, using the row's log-sum-exp saved by
//           the forward pass (the softmax is never normalised twice); D is written once, in bf16;
//   pass 2  dH = D W^T   (A = D, contraction over the vocabulary; both operands K-major);
//   pass 3  dW = H^T D   (A = H^T, contraction over the rows; both operands MN-major, read as stored).
// D is the only intermediate that touches HBM (M*V*2 bytes, written once and read by passes 2 and 3);
// the logits themselves never do. Given a mask, the rows with mask 0 (zero rows of D) are taken out of all three
// passes: H is packed first, D is written packed, and the kernels take the row count from the workspace header.
//
// Kernel structure (same as the forward kernel): one persistent block per SM, 192 threads: warp 0 = TMA
// producer (4-stage ring, 128-byte swizzle), warp 1 = tcgen05.mma issuer (M = 128, N = 256, K = 16 per
// instruction, fp32 accumulation in one of two 256-column tensor-memory buffers), warps 2-5 = epilogue
// (thread r owns row r of the tile, 32 columns per tcgen05.ld). Work unit = one 128 x 256 output tile
// with its whole contraction; units are ordered in groups of gm x gn tiles that run at the same time
// and share their operand panels through L2. Every wait is bounded (PPO_DEV_TIMEOUT on expiry).
#include "ppo_tcgen05.cuh"

namespace ppo {
namespace bwd {

constexpr int kBlockM = 128, kBlockN = 256, kBlockK = 64;
constexpr int kStages = 4;
constexpr int kABytes = kBlockM * kBlockK * 2;          // 16 KB
constexpr int kBoxBytes = 64 * kBlockK * 2;             // 8 KB: one 64 x 64 box of an MN-major operand
constexpr int kBBytes = kBlockN * kBlockK * 2;          // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;          // 48 KB
constexpr int kThreads = 192;

struct Smem {
    unsigned long long full[kStages], empty[kStages], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
};

using namespace tc;

struct Unit {
    int m_tile, n_tile;
};

// unit index -> output tile. Tiles are taken in blocks of gm x gn (m fastest inside a block), the
// blocks row-major over the tile grid; a block's tiles run at the same time on different SMs and
// read the same gm A-panels and gn B-panels.
__device__ __forceinline__ Unit unit_of(int u, int m_tiles, int n_tiles, int gm, int gn)
{
    const int bm = (m_tiles + gm - 1) / gm;            // blocks along m
    // walk the blocks; block (i, j) holds min(gm, m_tiles - i*gm) * min(gn, n_tiles - j*gn) tiles
    const int full_cols = n_tiles / gn, rem_n = n_tiles - full_cols * gn;
    int j = 0, base = 0;
    // tiles in one column of blocks (all bm blocks over m): m_tiles * width
    const int per_full_col = m_tiles * gn;
    j = u / per_full_col;
    if (j > full_cols) j = full_cols;
    if (j == full_cols && rem_n == 0) j = full_cols - 1;
    base = j * per_full_col;
    const int width = j < full_cols ? gn : rem_n;
    const int local = u - base;                          // inside this column of blocks
    const int per_block_full = gm * width;
    int i = local / per_block_full;
    if (i >= bm) i = bm - 1;
    const int height = min(gm, m_tiles - i * gm);
    const int l2 = local - i * per_block_full;           // inside the block: m fastest
    Unit r;
    r.m_tile = i * gm + l2 % height;
    r.n_tile = j * gn + l2 / height;
    return r;
}

struct Args {
    int Mdim, Ndim, Kc;          // output is [Mdim, Ndim], contraction length Kc
    int m_tiles, n_tiles, gm, gn, n_units;
    __nv_bfloat16 *out;          // [Mdim, Ndim], Ndim contiguous
    // pass 1 only: per-row inputs of the gradient epilogue
    const int32_t *tokens;
    const uint8_t *mask;         // nullable
    const float *lse;            // natural-log log-sum-exp of logits / tau, from the forward pass
    const float *g;              // gradient on the token log-probs
    float c, inv_tau;
    int *status;
    // Row packing (the call was given a mask): the rows dimension holds the rows with mask 1 only and their
    // number is known on the device: *dev_rows replaces Mdim (rows_role 1) or Kc (rows_role 2); the sizes above
    // are upper bounds. in_map: pass 1 reads its per-row inputs at in_map[row]; out_map: the output row of
    // packed row r is out_map[r].
    const int *dev_rows;
    int rows_role;
    const int32_t *in_map, *out_map;
};

// EPI 0: out = accumulator (bf16). EPI 1: out = g * (onehot - 2^(acc*c - Y)) / tau, Y = lse * log2(e).
template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const Args a)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ Smem sm;
    unsigned char *ring = smem_raw + ((1024u - (saddr(smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // every role walks the same unit list with the same contraction length
    int Mdim = a.Mdim, Kc = a.Kc, m_tiles = a.m_tiles, n_units = a.n_units;
    if (a.dev_rows) {
        const int n = max(0, min(*a.dev_rows, a.rows_role == 1 ? a.Mdim : a.Kc));
        if (a.rows_role == 1) {
            Mdim = n;
            m_tiles = (n + kBlockM - 1) / kBlockM;
            n_units = m_tiles * a.n_tiles;
        } else {
            Kc = n;
        }
    }
    const int k_blocks = (Kc + kBlockK - 1) / kBlockK;     // a ragged last block is zero-filled by the copies

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            barrier_init(&sm.full[s], 1);
            barrier_init(&sm.empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            barrier_init(&sm.tmem_full[b], 1);
            barrier_init(&sm.tmem_empty[b], 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_all(&sm.tmem_base);
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
                const Unit un = unit_of(u, m_tiles, a.n_tiles, a.gm, a.gn);
                const int m0 = un.m_tile * kBlockM, n0 = un.n_tile * kBlockN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    if (it >= kStages) wait(&sm.empty[s], ((it / kStages) - 1) & 1, a.status);
                    unsigned char *stage = ring + (size_t)s * kStageBytes;
                    barrier_expect_tx(&sm.full[s], (uint32_t)kStageBytes);
                    if (A_MN) {   // A stored [Kc, Mdim]: boxes of 64 (m) x 64 (k)
#pragma unroll
                        for (int j = 0; j < kBlockM / 64; ++j)
                            tma_load_2d(stage + j * kBoxBytes, &map_a, m0 + j * 64, kb * kBlockK, &sm.full[s]);
                    } else {      // A stored [Mdim, Kc]: one box of 64 (k) x 128 (m)
                        tma_load_2d(stage, &map_a, kb * kBlockK, m0, &sm.full[s]);
                    }
                    if (B_MN) {   // B stored [Kc, Ndim]: boxes of 64 (n) x 64 (k)
#pragma unroll
                        for (int j = 0; j < kBlockN / 64; ++j)
                            tma_load_2d(stage + kABytes + j * kBoxBytes, &map_b, n0 + j * 64, kb * kBlockK, &sm.full[s]);
                    } else {      // B stored [Ndim, Kc]: one box of 64 (k) x 256 (n)
                        tma_load_2d(stage + kABytes, &map_b, kb * kBlockK, n0, &sm.full[s]);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(A_MN, B_MN, kBlockM, kBlockN);
            uint32_t it = 0, tc = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x, ++tc) {
                const uint32_t buf = tc & 1;
                if (tc >= 2) wait(&sm.tmem_empty[buf], ((tc >> 1) - 1) & 1, a.status);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + buf * kBlockN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    wait(&sm.full[s], (it / kStages) & 1, a.status);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = saddr(ring + (size_t)s * kStageBytes);
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk) {
                        // K-major operand: 8-row groups 1024 B apart; 16 contraction elements = 32 bytes further.
                        // MN-major operand: 64-wide boxes 8192 B apart, 8 contraction rows 1024 B apart;
                        // 16 contraction rows = 2048 bytes further.
                        const uint64_t ad = A_MN ? smem_desc(a_addr + kk * 2048, kBoxBytes, 1024) : smem_desc(a_addr + kk * 32, 16, 1024);
                        const uint64_t bd = B_MN ? smem_desc(b_addr + kk * 2048, kBoxBytes, 1024) : smem_desc(b_addr + kk * 32, 16, 1024);
                        mma(tmem_d, ad, bd, idesc, (kb | kk) ? 1u : 0u);
                    }
                    commit(&sm.empty[s]);
                }
                commit(&sm.tmem_full[buf]);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        uint32_t tc = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x, ++tc) {
            const Unit un = unit_of(u, m_tiles, a.n_tiles, a.gm, a.gn);
            const int row = un.m_tile * kBlockM + row_in_tile;
            const bool row_ok = row < Mdim;
            // per-row scalars of the gradient epilogue
            int tok = -1;
            float gs = 0.f, off = 0.f;
            bool neg = false;
            const int src = (EPI == 1 && row_ok && a.in_map) ? a.in_map[row] : row;
            if (EPI == 1 && row_ok && (!a.mask || a.mask[src])) {
                tok = a.tokens[src];
                gs = a.g[src] * a.inv_tau;
                off = log2f(fabsf(gs)) - a.lse[src] * kLog2e;     // -gs * 2^(y - Y) = -+ 2^(y - Y + log2|gs|)
                neg = gs > 0.f;
            }
            const uint32_t buf = tc & 1;
            wait(&sm.tmem_full[buf], (tc >> 1) & 1, a.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + buf * kBlockN + ((uint32_t)(q * 32) << 16);
            __nv_bfloat16 *orow = a.out + (size_t)(row_ok ? (a.out_map ? a.out_map[row] : row) : 0) * a.Ndim;
#pragma unroll 1
            for (int cc = 0; cc < kBlockN / 32; ++cc) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld32(taddr + cc * 32, r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (cc == kBlockN / 32 - 1) {
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) barrier_arrive(&sm.tmem_empty[buf]);
                }
                const int col0 = un.n_tile * kBlockN + cc * 32;
                if (!row_ok || col0 >= a.Ndim) continue;
                float v[32];
                if (EPI == 1) {
                    if (gs == 0.f) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0.f;
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float e = ex2(fmaf(__uint_as_float(r[j]), a.c, off));
                            v[j] = neg ? -e : e;
                        }
                        if ((unsigned)(tok - col0) < 32u) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (tok - col0 == j) v[j] += gs;
                        }
                    }
                } else {
                    // (an empty contraction left the accumulator unwritten: the result is 0)
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = k_blocks > 0 ? __uint_as_float(r[j]) : 0.f;
                }
                // Ndim is a multiple of 8: whole 16-byte groups are inside or outside the row
#pragma unroll
                for (int j8 = 0; j8 < 4; ++j8) {
                    if (col0 + j8 * 8 < a.Ndim) {
                        uint4 w;
                        __nv_bfloat162 h;
                        h = __floats2bfloat162_rn(v[j8 * 8 + 0], v[j8 * 8 + 1]); w.x = *reinterpret_cast<uint32_t *>(&h);
                        h = __floats2bfloat162_rn(v[j8 * 8 + 2], v[j8 * 8 + 3]); w.y = *reinterpret_cast<uint32_t *>(&h);
                        h = __floats2bfloat162_rn(v[j8 * 8 + 4], v[j8 * 8 + 5]); w.z = *reinterpret_cast<uint32_t *>(&h);
                        h = __floats2bfloat162_rn(v[j8 * 8 + 6], v[j8 * 8 + 7]); w.w = *reinterpret_cast<uint32_t *>(&h);
                        *reinterpret_cast<uint4 *>(orow + col0 + j8 * 8) = w;
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem_free_all(tmem_base);
    }
}

// ---------------------------------------------------------------- host side
// zero rows [*n, next multiple of 128) of a [M, row16 * 16 bytes] matrix (at most 127 rows, none beyond M)
__global__ void __launch_bounds__(256)
zero_tail_rows_kernel(uint4 *__restrict__ base, int row16, const int *__restrict__ n, int M)
{
    const int rows = max(0, min(*n, M));
    const int j = rows + blockIdx.x;
    if (j >= M || j >= ((rows + kBlockM - 1) / kBlockM) * kBlockM) return;
    uint4 *dst = base + (size_t)j * row16;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (int i = threadIdx.x; i < row16; i += blockDim.x) dst[i] = z;
}

template <bool A_MN, bool B_MN, int EPI>
static int launch_gemm(const CUtensorMap &ma, const CUtensorMap &mb, Args a, int gm, int gn, cudaStream_t s)
{
    a.m_tiles = (a.Mdim + kBlockM - 1) / kBlockM;
    a.n_tiles = (a.Ndim + kBlockN - 1) / kBlockN;
    a.gm = gm;
    a.gn = gn;
    const int64_t units = (int64_t)a.m_tiles * a.n_tiles;
    if (units >= ((int64_t)1 << 31)) return PPO_ERR_SHAPE;
    a.n_units = (int)units;
    int dev = 0, sms = 148;
    PPO_RETURN_IF_CUDA(cudaGetDevice(&dev));
    PPO_RETURN_IF_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const size_t smem = (size_t)kStages * kStageBytes + 1024;
    auto kern = gemm_kernel<A_MN, B_MN, EPI>;
    PPO_RETURN_IF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = a.n_units < sms ? a.n_units : sms;
    kern<<<grid, kThreads, smem, s>>>(ma, mb, a);
    return launch_status();
}

}   // namespace bwd
}   // namespace ppo

using namespace ppo;

extern "C" int ppo_lmhead_bwd(const void *H, const void *W, int64_t M, int64_t K, int64_t V, const int32_t *tokens,
                              const uint8_t *mask, const float *lse, const float *dlogprob, float temperature,
                              void *dlogits, void *dH, void *dW, void *workspace, void *stream)
{
    if (M <= 0 || K <= 0 || V <= 0 || M >= ((int64_t)1 << 31) - 256 || V >= ((int64_t)1 << 31) - 256 ||
        K >= ((int64_t)1 << 31) - 256)
        return PPO_ERR_SHAPE;
    if (!(temperature > 0.f) || !finite_f(temperature)) return PPO_ERR_PARAM;
    if (!H || !W || !tokens || !lse || !dlogprob || !dlogits || !workspace) return PPO_ERR_NULL;
    // 16-byte row pitches for every operand in both roles: H [M,K], W [K,V], D [M,V]
    if (K % 8 != 0 || V % 8 != 0) return PPO_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(H) % 16 || reinterpret_cast<uintptr_t>(W) % 16 ||
        reinterpret_cast<uintptr_t>(dlogits) % 16 || reinterpret_cast<uintptr_t>(dH) % 16 ||
        reinterpret_cast<uintptr_t>(dW) % 16 || reinterpret_cast<uintptr_t>(workspace) % 256)
        return PPO_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int *status = &ws_header(workspace)->status;
    CUtensorMap ma, mb;
    int rc;
    bwd::Args a = {};
    a.status = status;

    // With a mask (and more than one row tile) the rows with mask 0 are taken out of all three passes: the other
    // rows of H are packed into the workspace, pass 1 writes their gradient rows packed at the front of dlogits
    // (its per-row inputs are read through the row order), pass 2 writes each row of dH at its original place
    // (dH is cleared first) and pass 3 contracts over the packed rows only. Their number is known on the device:
    // the kernels read it from the workspace header. Rows of the packed H and D between that number and the next
    // multiple of 128 are zero-filled, so the last contraction block of pass 3 adds nothing.
    const bool packed = mask && M > bwd::kBlockM;
    const int *n_rows = nullptr;
    const int32_t *order = nullptr;
    const void *Hp = H;
    if (packed) {
        const LmWorkspace lay = lm_workspace(M, K, V);
        rc = launch_lm_pack_rows(H, M, K, mask, workspace, lay, s);
        if (rc) return rc;
        unsigned char *ws = reinterpret_cast<unsigned char *>(workspace);
        n_rows = &ws_header(workspace)->n_tokens;
        order = reinterpret_cast<const int32_t *>(ws + lay.order_off);
        Hp = ws + lay.packed_off;
        bwd::zero_tail_rows_kernel<<<bwd::kBlockM, 256, 0, s>>>(reinterpret_cast<uint4 *>(dlogits), (int)(V / 8), n_rows,
                                                              (int)M);
        rc = launch_status();
        if (rc) return rc;
        if (dH) PPO_RETURN_IF_CUDA(cudaMemsetAsync(dH, 0, (size_t)M * (size_t)K * 2, s));
    }

    // pass 1: D = epilogue(H W): A = H [M,K] K-major, B = W [K,V] MN-major
    rc = bwd::make_map(&ma, Hp, (uint64_t)K, (uint64_t)M, bwd::kBlockM);
    if (rc) return rc;
    rc = bwd::make_map(&mb, W, (uint64_t)V, (uint64_t)K, 64);
    if (rc) return rc;
    a.Mdim = (int)M; a.Ndim = (int)V; a.Kc = (int)K;
    a.out = reinterpret_cast<__nv_bfloat16 *>(dlogits);
    a.tokens = tokens; a.mask = mask; a.lse = lse; a.g = dlogprob;
    a.c = kLog2e / temperature; a.inv_tau = 1.0f / temperature;
    a.dev_rows = n_rows; a.rows_role = 1; a.in_map = order; a.out_map = nullptr;
    rc = bwd::launch_gemm<false, true, 1>(ma, mb, a, 37, 4, s);
    if (rc) return rc;
    a.in_map = nullptr;

    if (dH) {   // pass 2: dH [M,K] = D [M,V] . W[K,V]^T: A = D K-major, B = W K-major; contraction over V
        rc = bwd::make_map(&ma, dlogits, (uint64_t)V, (uint64_t)M, bwd::kBlockM);
        if (rc) return rc;
        rc = bwd::make_map(&mb, W, (uint64_t)V, (uint64_t)K, bwd::kBlockN);
        if (rc) return rc;
        a.Mdim = (int)M; a.Ndim = (int)K; a.Kc = (int)V;
        a.out = reinterpret_cast<__nv_bfloat16 *>(dH);
        a.out_map = order;
        rc = bwd::launch_gemm<false, false, 0>(ma, mb, a, 37, 4, s);
        if (rc) return rc;
        a.out_map = nullptr;
    }
    if (dW) {   // pass 3: dW [K,V] = H[M,K]^T . D [M,V]: A = H MN-major, B = D MN-major; contraction over M
        rc = bwd::make_map(&ma, Hp, (uint64_t)K, (uint64_t)M, 64);
        if (rc) return rc;
        rc = bwd::make_map(&mb, dlogits, (uint64_t)V, (uint64_t)M, 64);
        if (rc) return rc;
        a.Mdim = (int)K; a.Ndim = (int)V; a.Kc = (int)M;
        a.out = reinterpret_cast<__nv_bfloat16 *>(dW);
        a.rows_role = 2;
        rc = bwd::launch_gemm<true, true, 0>(ma, mb, a, 8, 18, s);
        if (rc) return rc;
    }
    return PPO_OK;
}
