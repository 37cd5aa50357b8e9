// Tensor-core input projection for bf16 storage: G[m][n] = sum_k X[m][k] Wx[n][k] (+ bias[n]), the x_t
// half of W [x_t, h_{t-1}] + b of the paper's Section 4 cell equations for all timesteps at once.
//
// Blackwell-native structure: one CTA per (128 weight rows) x (n_tile activation rows) x (K split)
// output tile.  Both operands are K-major bf16 and arrive through TMA (cp.async.bulk.tensor, 128-byte
// swizzle, out-of-bounds rows and the K tail zero-filled) into a multi-stage shared-memory ring guarded
// by mbarriers; one elected thread issues tcgen05.mma (M = 128, N = n_tile, K = 16 per instruction)
// accumulating in tensor memory; four warps read the accumulator back with tcgen05.ld and store it with
// the bias.  Activations are fed as two bf16 terms (x = hi + lo, lo = bf16(x - hi)): each weight tile
// staged in shared memory is multiplied by both, so activations keep about 16 mantissa bits while the
// weights -- exactly bf16 -- are read only once.  The weights are the M operand, so a short sequence
// (T*B = 35) still fills the MMA's 128-row dimension; such weight-read-bound shapes are split along K
// over otherwise idle SMs and the partial planes are added up by the recurrent kernel.  No TMA multicast is used: each CTA fetches its
// own tiles.  Every mbarrier wait is bounded; on expiry the kernel records a timeout status, and all
// roles fall through to the common exit where tensor memory is released.
#include "common.cuh"
#include "device_util.cuh"

#include <cuda.h>
#include <cstdio>
#include <cstring>
#include <cstdlib>

namespace lstm {
namespace {

constexpr int kBM = 128;          // weight rows per tile (MMA M)
constexpr int kBK = 64;           // K elements per stage: 128 bytes of bf16 = one swizzle atom row
constexpr int kThreads = 192;     // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr int kMaxStages = 8;
constexpr int kMaxNTile = 128;    // activation rows per tile (MMA N); two activation tiles (hi, lo) per stage

struct TcArgs {
    int M, N, K;
    int n_tile, nsplit, kblocks, stages, tmem_cols;
    float *G;
    const float *bias;
    int *status;
    long long g_split_stride;
};






__global__ void __launch_bounds__(kThreads, 2)
proj_tc_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
               const __grid_constant__ CUtensorMap tmap_xlo, const TcArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[kMaxStages], empty_bar[kMaxStages], accum_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int w_tile = blockIdx.x, x_tile = blockIdx.y, split = blockIdx.z;
    const int kb0 = (int)((long long)split * a.kblocks / a.nsplit);
    const int kb1 = (int)((long long)(split + 1) * a.kblocks / a.nsplit);
    const int nkb = kb1 - kb0;
    const int S = a.stages;
    const uint32_t a_bytes = kBM * kBK * 2, b_bytes = (uint32_t)a.n_tile * kBK * 2;
    const uint32_t stage_bytes = a_bytes + 2 * b_bytes;                 // weights, x hi, x lo; multiple of 1024
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;      // swizzled tiles need 1024-byte alignment

    if (tid == 0) {
        abort_s = 0;
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        mbar_init(smem_u32(&accum_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    volatile int *abort_flag = &abort_s;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer
            int s = 0;
            uint32_t ph = 0;
            for (int i = 0; i < nkb; ++i) {
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag)) break;
                const uint32_t fb = smem_u32(&full_bar[s]);
                mbar_expect_tx(fb, stage_bytes);
                const uint32_t sa = tiles + (uint32_t)s * stage_bytes;
                tma_load_2d(sa, &tmap_w, fb, (kb0 + i) * kBK, w_tile * kBM);
                tma_load_2d(sa + a_bytes, &tmap_x, fb, (kb0 + i) * kBK, x_tile * a.n_tile);
                tma_load_2d(sa + a_bytes + b_bytes, &tmap_xlo, fb, (kb0 + i) * kBK, x_tile * a.n_tile);
                if (++s == S) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer
            // instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, M = 128, N = 2 * n_tile: the
            // hi and the lo activation tiles lie back to back in the stage and form ONE operand of 2 * n_tile
            // rows (an instruction of this size costs the same whatever N, so one is half the price of two);
            // accumulator columns [0, n_tile) hold the hi product, [n_tile, 2 n_tile) the lo product
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * a.n_tile) >> 3) << 17) |
                                   ((uint32_t)(kBM >> 4) << 24);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int i = 0; i < nkb && ok; ++i) {
                ok = mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = tiles + (uint32_t)s * stage_bytes;
                const uint64_t adesc = umma_desc_sw128(sa), bdesc = umma_desc_sw128(sa + a_bytes);
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k)
                    umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                umma_commit(smem_u32(&empty_bar[s]));      // frees the stage once these MMAs have read it
                if (++s == S) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(smem_u32(&accum_bar));     // accumulator complete
        }
    } else {
        // ---- epilogue: warp w may touch TMEM lanes 32*(w % 4) .. +31
        const int lq = warp & 3;
        const bool ok = mbar_wait(smem_u32(&accum_bar), 0u, abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            const int n = w_tile * kBM + lq * 32 + lane;                  // weight row = G column
            const float bv = (split == 0 && a.bias && n < a.N) ? a.bias[n] : 0.0f;
            float *gout = a.G + (size_t)split * a.g_split_stride;
            for (int c0 = 0; c0 < a.n_tile; c0 += 16) {
                uint32_t v[16], vlo[16];
                tmem_ld16(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0, v);
                tmem_ld16(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(a.n_tile + c0), vlo);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int m0 = x_tile * a.n_tile + c0;
                if (n < a.N) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (m0 + i < a.M) gout[(size_t)(m0 + i) * a.N + n] = __uint_as_float(v[i]) + __uint_as_float(vlo[i]) + bv;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
    if (tid == 0 && abort_s) atomicExch(a.status, kStatusTimeout);
}

// Tensor-bound shapes (several activation tiles): a persistent kernel, one CTA per SM, whose tile is 256 weight
// rows x n_tile activation rows: two M = 128 accumulators share each staged activation tile, so a K block costs
// 32 KB of weights + 2 x n_tile x 128 B of activations for twice the products of the kernel above (whose 128-row
// tile asks L2 for more bytes per product than it delivers to 148 SMs at once).  The producer keeps fetching
// the next tile's stages while the four read-back warps store the finished one; the issuing thread waits for
// them to leave tensor memory (a second barrier) before it overwrites the accumulators.
struct TcBigArgs {
    int M, N, K;
    int n_tile, kblocks, stages, tmem_cols;
    int wtiles, xtiles;            // 256-row weight tiles, activation tiles
    float *G;
    const float *bias;
    int *status;
};

__global__ void __launch_bounds__(kThreads, 1)
proj_tc_big_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                   const __grid_constant__ CUtensorMap tmap_xlo, const TcBigArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[kMaxStages], empty_bar[kMaxStages], accum_bar, drained_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = a.stages, nkb = a.kblocks;
    const int ntiles = a.wtiles * a.xtiles;
    const uint32_t a_bytes = kBM * kBK * 2, b_bytes = (uint32_t)a.n_tile * kBK * 2;
    const uint32_t stage_bytes = 2 * a_bytes + 2 * b_bytes;             // two weight tiles, x hi, x lo; multiple of 1024
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    LSTM_CHECK_SMEM_END((size_t)(tiles - smem_u32(smem_raw)) + (size_t)S * stage_bytes, a.status);

    if (tid == 0) {
        abort_s = 0;
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        mbar_init(smem_u32(&accum_bar), 1);
        mbar_init(smem_u32(&drained_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    volatile int *abort_flag = &abort_s;
    // consecutive CTAs take tiles that share the activation tile (x_tile slow, w_tile fast): they are in L2 together
    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer: runs ahead of the MMA thread by up to S stages, across tile boundaries
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int w_tile = tile % a.wtiles, x_tile = tile / a.wtiles;
                for (int i = 0; i < nkb; ++i) {
                    ok = mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t fb = smem_u32(&full_bar[s]);
                    mbar_expect_tx(fb, stage_bytes);
                    const uint32_t sa = tiles + (uint32_t)s * stage_bytes;
                    tma_load_2d(sa, &tmap_w, fb, i * kBK, w_tile * 2 * kBM);
                    tma_load_2d(sa + a_bytes, &tmap_w, fb, i * kBK, w_tile * 2 * kBM + kBM);     // may lie beyond N: zero fill
                    tma_load_2d(sa + 2 * a_bytes, &tmap_x, fb, i * kBK, x_tile * a.n_tile);
                    tma_load_2d(sa + 2 * a_bytes + b_bytes, &tmap_xlo, fb, i * kBK, x_tile * a.n_tile);
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer: accumulator h (weight rows h*128 .. +127 of the tile) at TMEM column h * 2 * n_tile;
            // columns [0, n_tile) of an accumulator hold the hi product, [n_tile, 2 n_tile) the lo product
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * a.n_tile) >> 3) << 17) |
                                   ((uint32_t)(kBM >> 4) << 24);
            const uint32_t acc1 = tmem_base + (uint32_t)(2 * a.n_tile);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0, tph = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, tph ^= 1u) {
                // the read-back warps have left the accumulators of the previous tile
                ok = mbar_wait(smem_u32(&drained_bar), tph ^ 1u, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int i = 0; i < nkb && ok; ++i) {
                    ok = mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = tiles + (uint32_t)s * stage_bytes;
                    const uint64_t adesc0 = umma_desc_sw128(sa), adesc1 = umma_desc_sw128(sa + a_bytes);
                    const uint64_t bdesc = umma_desc_sw128(sa + 2 * a_bytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        umma_bf16(tmem_base, adesc0 + 2 * k, bdesc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                        umma_bf16(acc1, adesc1 + 2 * k, bdesc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&empty_bar[s]));
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&accum_bar));
            }
        }
    } else {
        // ---- read-back: warp w may touch TMEM lanes 32*(w % 4) .. +31; thread = one weight row = one G column
        const int lq = warp & 3;
        uint32_t tph = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, tph ^= 1u) {
            const bool ok = mbar_wait(smem_u32(&accum_bar), tph, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int w_tile = tile % a.wtiles, x_tile = tile / a.wtiles;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                const int n = w_tile * 2 * kBM + half * kBM + lq * 32 + lane;
                const float bv = (a.bias && n < a.N) ? a.bias[n] : 0.0f;
                const uint32_t acc = tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(half * 2 * a.n_tile);
                for (int c0 = 0; c0 < a.n_tile; c0 += 16) {
                    uint32_t v[16], vlo[16];
                    tmem_ld16(acc + (uint32_t)c0, v);
                    tmem_ld16(acc + (uint32_t)(a.n_tile + c0), vlo);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int m0 = x_tile * a.n_tile + c0;
                    if (n < a.N) {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (m0 + i < a.M) a.G[(size_t)(m0 + i) * a.N + n] = __uint_as_float(v[i]) + __uint_as_float(vlo[i]) + bv;
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            bar_sync(1, 128);
            if (tid == 64) mbar_arrive(smem_u32(&drained_bar));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
    if (tid == 0 && abort_s) atomicExch(a.status, kStatusTimeout);
}
// rows x K bf16 matrix with row stride ldk elements; box = 64 x box_rows, 128-byte swizzle, zero fill
bool encode_2d(CUtensorMap *map, const void *base, int rows, int K, int ldk, int box_rows)
{
    return encode_tmap_bf16_2d(map, base, rows, K, ldk, box_rows);
}

constexpr int kSmemBudget = 200 * 1024;

}  // namespace

static_assert(sizeof(CUtensorMap) == 128, "tensor map size");

int proj_tc_plan(ProjTcPlan *p, const __nv_bfloat16 *W, const __nv_bfloat16 *X, const __nv_bfloat16 *Xlo,
                 int M, int N, int K, int ldk, int sm_count, char *err, int errlen)
{
    if (M < 1 || N < 1 || K < 1 || (ldk % 8) != 0 || ((uintptr_t)W & 15) || ((uintptr_t)X & 15) || ((uintptr_t)Xlo & 15)) {
        snprintf(err, errlen, "operands must be 16-byte aligned with row strides that are multiples of 8 elements");
        return 1;
    }
    memset(p, 0, sizeof *p);
    p->M = M; p->N = N; p->K = K; p->ldk = ldk; p->sm_count = sm_count;
    p->kblocks = (K + kBK - 1) / kBK;
    const int wtiles = (N + kBM - 1) / kBM;
    int xtiles = (M + kMaxNTile - 1) / kMaxNTile;
    int n_tile = ((M + xtiles - 1) / xtiles + 15) / 16 * 16;
    if (n_tile > kMaxNTile) n_tile = kMaxNTile;
    xtiles = (M + n_tile - 1) / n_tile;
    p->n_tile = n_tile;
    // weight-read-bound shapes (a single activation tile): split K over SMs that would otherwise idle
    int nsplit = 1;
    if (xtiles == 1) {
        nsplit = sm_count / wtiles;
        if (nsplit > 4) nsplit = 4;
        if (nsplit > p->kblocks) nsplit = p->kblocks;
        if (nsplit < 1) nsplit = 1;
    }
    p->nsplit = nsplit;
    if (!encode_2d(reinterpret_cast<CUtensorMap *>(p->tmap_w), W, N, K, ldk, kBM) ||
        !encode_2d(reinterpret_cast<CUtensorMap *>(p->tmap_x), X, M, K, ldk, n_tile) ||
        !encode_2d(reinterpret_cast<CUtensorMap *>(p->tmap_xlo), Xlo, M, K, ldk, n_tile)) {
        snprintf(err, errlen, "cuTensorMapEncodeTiled failed (N=%d M=%d K=%d ldk=%d n_tile=%d)", N, M, K, ldk, n_tile);
        return 1;
    }
    return 0;
}

cudaError_t proj_tc_prepare()
{
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(proj_tc_big_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024);
    if (e != cudaSuccess) return e;
    // two CTAs of half the budget share an SM: ask for the largest shared-memory carve-out
    return cudaFuncSetAttribute(proj_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}

cudaError_t launch_proj_tc(const ProjTcPlan &p, const float *bias, float *G, int *status, cudaStream_t st)
{
    const int xt = (p.M + p.n_tile - 1) / p.n_tile;
    const char *tile_env = getenv("LSTM_B200_PROJ_TILE");
    if (xt > 1 && p.nsplit == 1 && !(tile_env && atoi(tile_env) == 128)) {
        // several activation tiles: the persistent kernel with 256-row weight tiles
        TcBigArgs b;
        b.M = p.M; b.N = p.N; b.K = p.K;
        b.n_tile = p.n_tile; b.kblocks = p.kblocks;
        const int stage_bytes = 2 * kBM * kBK * 2 + 2 * p.n_tile * kBK * 2;
        int stages = kSmemBudget / stage_bytes;
        if (stages > kMaxStages) stages = kMaxStages;
        b.stages = stages;
        int cols = 32;
        while (cols < 4 * p.n_tile) cols <<= 1;      // two accumulators, hi and lo products side by side in each
        b.tmem_cols = cols;
        b.wtiles = (p.N + 2 * kBM - 1) / (2 * kBM);
        b.xtiles = xt;
        b.G = G; b.bias = bias; b.status = status;
        const int ntiles = b.wtiles * b.xtiles;
        const int grid = ntiles < p.sm_count ? ntiles : (p.sm_count > 0 ? p.sm_count : 1);
        const size_t smem = (size_t)stages * stage_bytes + 1024;
        proj_tc_big_kernel<<<grid, kThreads, smem, st>>>(*reinterpret_cast<const CUtensorMap *>(p.tmap_w),
                                                         *reinterpret_cast<const CUtensorMap *>(p.tmap_x),
                                                         *reinterpret_cast<const CUtensorMap *>(p.tmap_xlo), b);
        return cudaGetLastError();
    }
    TcArgs a;
    a.M = p.M; a.N = p.N; a.K = p.K;
    a.n_tile = p.n_tile; a.nsplit = p.nsplit; a.kblocks = p.kblocks;
    const int stage_bytes = kBM * kBK * 2 + 2 * p.n_tile * kBK * 2;
    // Many activation tiles (T*B large, tensor-bound): two CTAs per SM with two stages each, so that one CTA's
    // read-back and stores overlap the other's products; a single activation tile (weight-read-bound): one CTA
    // per SM with a deep ring.
    int budget = kSmemBudget;
    if ((p.M + p.n_tile - 1) / p.n_tile > 1) budget = kSmemBudget / 2;
    if (const char *e = getenv("LSTM_B200_PROJ_SMEM_KB")) { const int kb = atoi(e); if (kb >= 48 && kb <= 200) budget = kb * 1024; }
    int stages = budget / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    const int max_kb = (p.kblocks + p.nsplit - 1) / p.nsplit;
    if (stages > max_kb) stages = max_kb;
    if (stages < 1) stages = 1;
    a.stages = stages;
    int cols = 32;
    while (cols < 2 * p.n_tile) cols <<= 1;      // hi and lo products side by side
    a.tmem_cols = cols;
    a.G = G; a.bias = bias; a.status = status;
    a.g_split_stride = (long long)p.M * p.N;
    const int wtiles = (p.N + kBM - 1) / kBM;
    const int xtiles = (p.M + p.n_tile - 1) / p.n_tile;
    dim3 grid(wtiles, xtiles, p.nsplit);
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    proj_tc_kernel<<<grid, kThreads, smem, st>>>(*reinterpret_cast<const CUtensorMap *>(p.tmap_w),
                                                 *reinterpret_cast<const CUtensorMap *>(p.tmap_x),
                                                 *reinterpret_cast<const CUtensorMap *>(p.tmap_xlo), a);
    return cudaGetLastError();
}

}  // namespace lstm
