// Batched recurrent kernel for bf16 weights on the 5th-generation tensor cores: the serial half of the LSTM
// forward pass (paper, Section 4, cell equations with zero hidden layers per gate)
//     z = G[t] + Wh h_{t-1};  i,f,o = sigmoid(z_i,z_f,z_o), g = tanh(z_g);  c_t = f c_{t-1} + i g;
//     h_t = o tanh(c_t)
// for batches of five to kTcMaxBatch sequences, where the per-step product Wh_slice [4u x H] . h_{t-1} [H x B]
// is a real (if skinny) matrix product and one tcgen05.mma chain per step replaces the ceil(B/4) passes of
// the register-resident kernel.
//
// One cooperative launch runs all T steps of one layer (both directions on disjoint CTA groups).  A CTA
// owns a contiguous range of hidden units; its slice of Wh (rows 4*unit + gate) is loaded ONCE by TMA into
// shared memory as 128-byte-swizzled K-major tiles (one per 64 columns) and stays there.  h travels
// between CTAs through global memory as the tensor cores want it: two bf16 planes per batch row (row 2b =
// hi, row 2b+1 = lo, so products keep about 16 mantissa bits), K-major.  Per step:
//   warp 0   waits until its own CTA has published the previous step, polls one stamp per producer CTA
//            (relaxed loads, all in flight together, one fence after the last; bounded), then streams the
//            [2B x H] operand into a ring of shared-memory stages with TMA (up to four 64-column blocks per
//            stage, one issuing lane per block, zero fill at the tail).  Every CTA (pair) reads the whole
//            operand from L2, 148 SMs at once: this fetch, about 20 bytes per clock and SM, is the longest
//            single part of a step;
//   warps 1-3 issue M = 128, N = 2B (rounded up to 16), K = 16 tcgen05.mma instructions.  One thread issues
//            such an instruction every 70 cycles or so whatever its shape, while the tensor cores finish it
//            in far less at these N, so the K blocks are dealt round-robin to up to three issuing threads in
//            three warps, each with a TMEM accumulator of its own (measured for 48 instructions: 3400
//            cycles from one thread, 2340 from two, 1410 from four).  The weight tile has only 4*units
//            (<= 128) real rows: the rows beyond read whatever follows in shared memory and produce
//            accumulator rows nobody reads;
//   warps 4-7 request their projection terms, then read the accumulator rows of the CTA's units back
//            (tcgen05.ld), add the issuers' accumulators and the hi and lo columns, and finish the (unit,
//            batch row) pairs: gates, c/h update, outputs, and the new h as bf16 planes; then one thread
//            fences and raises the CTA's stamp.
// Pair mode (chosen at create time when the CTA count per direction is even, the doubled tile fits and the
// device can co-schedule the clusters): CTAs 2p and 2p+1 are launched as a cluster of two; each keeps the
// weight rows of BOTH CTAs' units but only half of the K blocks, so each issues half the tensor
// instructions per step; the partial sums of the partner's units are collected in shared memory and
// sent to the partner's with one bulk copy (cp.async.bulk shared::cta -> shared::cluster) that completes on the
// partner's mbarrier, and every CTA finishes its own units from its own and the received partial sums.  The wait for the partner is bounded like the rest,
// and a cluster barrier at the common exit keeps a CTA resident while its partner may still write into it.
// Every wait (stamps, mbarriers) is bounded; on expiry the CTA records a timeout status and all roles fall
// through to the common exit where tensor memory is released.  No TMA multicast is used.
#include "common.cuh"
#include "device_util.cuh"

#include <cuda.h>
#include <cstdio>
#include <cstring>

namespace lstm {
namespace {

constexpr int kThreads = 256;                  // producer warp, three issuing warps, four finishing warps
constexpr int kFinishTid0 = 128;                // first thread of the finishing warps
constexpr int kMaxStages = 8;
constexpr int kFlagLoads = 5;                   // stamps one lane polls: up to 160 CTAs per direction
constexpr int kPre = 2;                         // (unit, batch row) items per thread whose projection terms are prefetched
constexpr int kMaxSplit = 4;                    // split-K partial sums of the projection

// ---- two-CTA cluster helpers (pair mode): the partner's shared memory and barriers
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
// shared memory of this CTA -> shared memory of another CTA of the cluster (addresses and size multiples of 16
// bytes); the bytes are counted on the destination CTA's barrier
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t remote_dst, uint32_t local_src, uint32_t bytes, uint32_t remote_bar)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(remote_dst), "r"(local_src), "r"(bytes), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}


__global__ void __launch_bounds__(kThreads, 1)
recur_tc_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_h, const RecurTcArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[kMaxStages], empty_bar[kMaxStages], accum_bar, w_bar, partial_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, pub_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = a.H, B = a.B, T = a.T, D = a.D, N = a.N, S = a.stages, RA = a.RA, nkb = a.nkb, kbs = a.kbs;
    const int NB = (2 * B + 7) & ~7;             // rows of a fetched operand block: the copy leaves out the rows that only pad N
    const int d = a.dir0 + blockIdx.x / a.ncta_dir;
    const int cta = blockIdx.x % a.ncta_dir;
    int u0, nu;
    unit_range(H, a.ncta_dir, cta, u0, nu);
    const int upc = (H + a.ncta_dir - 1) / a.ncta_dir;
    // Pair mode: CTAs 2p and 2p+1 form a cluster; each keeps the rows of BOTH CTAs' units (RT = 2 RA rows) but
    // only half of the K blocks, multiplies its half, and hands the partner the partial sums of the partner's
    // units through distributed shared memory: half the tensor instructions per step and CTA.
    const int pair = a.pair;
    const int rank = pair ? (int)cluster_ctarank() : 0;
    const int RT = pair ? 2 * RA : RA;                                      // rows of a weight tile
    const int nkb_half = (nkb + 1) / 2;
    const int kb_lo = (pair && rank) ? nkb_half : 0;                        // first K block of this CTA
    const int nkb_my = pair ? (rank ? nkb - nkb_half : nkb_half) : nkb;     // K blocks of this CTA
    const int nkb_alloc = pair ? nkb_half : nkb;                            // same layout in both CTAs of a pair
    const int groups = (nkb_my + kbs - 1) / kbs;                            // ring stages one step's operand takes
    const bool whole = groups <= S && nkb_my <= 32;                         // the ring holds it all: every step starts at stage 0

    // shared-memory carve-up (tiles need 1024-byte alignment): weight tiles, operand ring, then scratch
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_tiles = base;                                          // [nkb_alloc][RT rows][128 B]
    const uint32_t ring = a_tiles + (uint32_t)nkb_alloc * RT * 128;         // [S][kbs][N rows][128 B]
    unsigned char *gen = smem_raw + (ring + (uint32_t)(S * kbs * N) * 128 - smem_u32(smem_raw));
    float *zs = reinterpret_cast<float *>(gen);                             // [B][4*upc] gate pre-activations (h part)
    const int zld = 4 * upc;
    float *c_s = zs + zld * B;                                              // [B][units of this CTA]
    float *zs2 = c_s + ((upc * B + 3) & ~3);                                // [B][4*upc] partial sums received from the partner (pair mode)
    float *zsp = zs2 + (pair ? zld * B : 0);                                // [B][4*upc] partial sums of the partner's units, before they are sent
    // checked build: the carve-up ends inside the launch's shared memory, and so does the 128-row read of the last weight tile
    LSTM_CHECK_SMEM_END((size_t)(reinterpret_cast<unsigned char *>(zsp + (pair ? zld * B : 0)) - smem_raw), a.status);
    LSTM_CHECK_SMEM_END((size_t)(a_tiles - smem_u32(smem_raw)) + (size_t)(nkb_alloc - 1) * RT * 128 + (size_t)128 * 128, a.status);

    if (tid == 0) {
        abort_s = 0;
        pub_s = 0;
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), (uint32_t)a.nissue); }
        mbar_init(smem_u32(&accum_bar), (uint32_t)a.nissue);
        mbar_init(smem_u32(&w_bar), 1);
        mbar_init(smem_u32(&partial_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (int i = tid; i < nu * B; i += kThreads) {
        const int b = i / nu, u = i - b * nu;
        c_s[i] = a.c0 ? a.c0[((size_t)d * B + b) * H + u0 + u] : 0.0f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (pair) cluster_sync_all();               // the partner's barriers are initialised before anything reaches them
    const uint32_t tmem_base = tmem_base_s;
    volatile int *abort_flag = &abort_s;
    volatile int *pub = &pub_s;                 // steps this CTA has published (h0 counts as one)

    __nv_bfloat16 *hbuf_d = a.hbuf + (size_t)d * 2 * kTcPlaneRows * a.ldh;  // [parity][kTcPlaneRows rows][ldh]
    unsigned *flags_d = a.flags + (size_t)d * a.ncta_dir;

    if (warp == 0) {
        // ================= stamps and TMA =================
        // the CTA's weight tiles, once (one lane per tile)
        if (lane == 0) mbar_expect_tx(smem_u32(&w_bar), (uint32_t)nkb_my * RT * 128);
        __syncwarp();
        for (int kb = lane; kb < nkb_my; kb += 32)
            tma_load_2d(a_tiles + (uint32_t)kb * RT * 128, &tmap_w, smem_u32(&w_bar), (kb_lo + kb) * 64,
                        (d * a.ncta_dir + (pair ? (cta & ~1) : cta)) * RA);
        // ring position as a stage index and a phase bit (a 64-bit divide per stage would cost the issuing
        // thread more than the copies it issues)
        int st = 0;
        uint32_t ph = 0;
        bool live = true;
        for (int s = 0; s < T && live; ++s) {
            // Do not poll before this CTA has published its own part of the previous step: loads that spin
            // ahead of the data queue up in front of the SM's own stores and delay every consumer.
            if (lane == 0) {
                long long t_start = 0;
                for (int it = 0; *pub < s + 1; ++it) {
                    if ((it & 63) == 63) {
                        const long long now = clock64();
                        if (t_start == 0) t_start = now;
                        if (now - t_start > a.spin_limit || *abort_flag) { *abort_flag = 1; break; }
                    }
                }
            }
            __syncwarp();
            // every producer's stamp of the previous step (the prologue publishes h0 with stamp_base): relaxed
            // loads, all in flight together, and one fence once they all show the stamp (acquire loads in the
            // polling loop were measured far slower)
            const unsigned want = a.stamp_base + (unsigned)s;
            long long t_start = 0;
            int rounds = 0;
            bool aborted = false;
            bool seen[kFlagLoads];
#pragma unroll
            for (int k = 0; k < kFlagLoads; ++k) seen[k] = lane + 32 * k >= a.ncta_dir;
            while (true) {
                // only the stamps not yet seen are asked for again: most producers are early, and the lines
                // that hold the stamps are the busiest in the L2 (every CTA reads and writes them)
                unsigned v[kFlagLoads];
#pragma unroll
                for (int k = 0; k < kFlagLoads; ++k)
                    if (!seen[k]) v[k] = ld_relaxed_u32(flags_d + lane + 32 * k);
                bool ok = true;
#pragma unroll
                for (int k = 0; k < kFlagLoads; ++k) {
                    if (!seen[k]) seen[k] = (int)(v[k] - want) >= 0;
                    ok &= seen[k];
                }
                // both votes are taken by all lanes every round, so the warp leaves the loop as one
                if (__any_sync(0xffffffffu, *abort_flag != 0)) { aborted = true; break; }
                if (__all_sync(0xffffffffu, ok)) break;
                if ((++rounds & 15) == 0) {
                    const long long now = clock64();
                    if (t_start == 0) t_start = now;
                    if (now - t_start > a.spin_limit || ld_volatile_s32(a.status) != kStatusOk) *abort_flag = 1;
                }
            }
            if (aborted) break;
            fence_acq_rel_gpu();                                    // acquire: the planes behind the stamps
            asm volatile("fence.proxy.async.global;" ::: "memory");    // they were written with ordinary stores
            const int row0 = (d * 2 + ((s + 1) & 1)) * kTcPlaneRows;   // planes of step s-1 live in parity (s-1)&1
            if (whole) {
                // the ring holds the whole operand (every step starts at stage 0 with the same phase): lane i < groups
                // opens stage i, then one lane per K block issues its copy, all in the same instruction
                int ok = 1;
                if (lane < groups) {
                    const int nblk = min(kbs, nkb_my - lane * kbs);
                    ok = mbar_wait(smem_u32(&empty_bar[lane]), ((uint32_t)s & 1u) ^ 1u, abort_flag) ? 1 : 0;
                    if (ok) mbar_expect_tx(smem_u32(&full_bar[lane]), (uint32_t)(nblk * NB) * 128);
                }
                if (!__all_sync(0xffffffffu, ok)) break;
                if (lane < nkb_my)
                    tma_load_2d(ring + (uint32_t)(lane * N) * 128, &tmap_h, smem_u32(&full_bar[lane / kbs]), (kb_lo + lane) * 64, row0);
                continue;
            }
            for (int g0 = 0; g0 < nkb_my; g0 += kbs) {
                const int nblk = min(kbs, nkb_my - g0);
                int ok = 1;
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&empty_bar[st]), ph ^ 1u, abort_flag) ? 1 : 0;
                    if (ok) mbar_expect_tx(smem_u32(&full_bar[st]), (uint32_t)(nblk * NB) * 128);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { live = false; break; }
                // one lane per K block of the stage: issuing a tensor copy occupies a thread for a while
                if (lane < nblk)
                    tma_load_2d(ring + (uint32_t)((st * kbs + lane) * N) * 128, &tmap_h, smem_u32(&full_bar[st]), (kb_lo + g0 + lane) * 64, row0);
                if (++st == S) { st = 0; ph ^= 1u; }
            }
        }
    } else if (warp <= 3) {
        // ================= MMA issue =================
        // issuer w = warp - 1 < nissue takes the K blocks whose index is w modulo nissue (no CTA has fewer K blocks
        // than issuers) into the accumulator at TMEM column w * N; every issuer passes every stage and commits to
        // its barriers, blocks or not
        const int w = warp - 1;
        if (lane == 0 && w < a.nissue) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            bool ok = mbar_wait(smem_u32(&w_bar), 0u, abort_flag);
            // descriptors differ only in their start-address field (units of 16 bytes): build one of each and add
            const uint64_t adesc0 = umma_desc_sw128(a_tiles), bdesc0 = umma_desc_sw128(ring);
            const uint32_t a_step = (uint32_t)(RT * 128) >> 4, b_step = (uint32_t)(N * 128) >> 4;
            const uint32_t acc = tmem_base + (uint32_t)(w * N);
            int st = 0;
            uint32_t ph = 0;
            for (int s = 0; s < T && ok; ++s) {
                uint32_t accumulate = 0u;
                int next = w;                                   // this issuer's next K block
                if (whole) { st = 0; ph = (uint32_t)s & 1u; }
                for (int g0 = 0; g0 < nkb_my; g0 += kbs) {
                    const int nblk = min(kbs, nkb_my - g0);
                    ok = mbar_wait(smem_u32(&full_bar[st]), ph, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    for (; next < g0 + nblk; next += a.nissue) {
                        const int l = next - g0;
                        const uint64_t adesc = adesc0 + (uint64_t)((uint32_t)(g0 + l) * a_step);
                        const uint64_t bdesc = bdesc0 + (uint64_t)((uint32_t)(st * kbs + l) * b_step);
                        umma_bf16(acc, adesc, bdesc, idesc, accumulate);
                        umma_bf16(acc, adesc + 2, bdesc + 2, idesc, 1u);
                        umma_bf16(acc, adesc + 4, bdesc + 4, idesc, 1u);
                        umma_bf16(acc, adesc + 6, bdesc + 6, idesc, 1u);
                        accumulate = 1u;
                    }
                    umma_commit(smem_u32(&empty_bar[st]));
                    if (++st == S) { st = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&accum_bar));
            }
        }
    } else {
        // ================= accumulator read-back and the cell =================
        const int ftid = tid - kFinishTid0;              // 0..127
        const int lq = warp & 3;                         // TMEM lane quadrant this warp may read
        const int nuB = nu * B;
        int u0_partner = 0, nu_partner = 0;
        uint32_t zs2_remote = 0, partial_bar_remote = 0;
        if (pair) {
            unit_range(H, a.ncta_dir, cta ^ 1, u0_partner, nu_partner);
            zs2_remote = map_to_cta(smem_u32(zs2), (uint32_t)(rank ^ 1));
            partial_bar_remote = map_to_cta(smem_u32(&partial_bar), (uint32_t)(rank ^ 1));
        }
        // the planes of h0 (stamp_base): this CTA's units
        for (int p = ftid; p < nuB; p += 128) {
            const int b = p / nu, u = p - b * nu;
            const float v = a.h0 ? a.h0[((size_t)d * B + b) * H + u0 + u] : 0.0f;
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            __nv_bfloat16 *row = hbuf_d + ((size_t)1 * kTcPlaneRows + 2 * b) * a.ldh + u0 + u;     // step -1 -> parity 1
            row[0] = hi;
            row[a.ldh] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
        bar_sync(1, 128);
        if (ftid == 0) {
            if ((int)blockIdx.x != a.withhold_cta) {
                fence_acq_rel_gpu();
                st_relaxed_u32(flags_d + cta, a.stamp_base);
            }
            *pub = 1;
        }
        const size_t gs4 = (size_t)(a.g_split_stride / 4);
        // the first kPre items of this thread: batch row and unit, fixed for the whole sequence
        int pb[kPre], pu[kPre];
#pragma unroll
        for (int i = 0; i < kPre; ++i) {
            const int p = ftid + 128 * i;
            pb[i] = p < nuB ? p / nu : 0;
            pu[i] = p < nuB ? p - pb[i] * nu : 0;
        }
        for (int s = 0; s < T; ++s) {
            const int t = d ? (T - 1 - s) : s;
            // projection terms of the first items: requested before the wait, they do not depend on h
            float4 gpre[kPre][kMaxSplit];
#pragma unroll
            for (int i = 0; i < kPre; ++i) {
                const int p = ftid + 128 * i;
                if (p < nuB) {
                    const int b = pb[i], j = u0 + pu[i];
                    const float4 *gp = reinterpret_cast<const float4 *>(a.G + (((size_t)t * B + b) * D + d) * 4 * H + (size_t)j * 4);
#pragma unroll
                    for (int sp = 0; sp < kMaxSplit; ++sp)
                        if (sp < a.nsplit) gpre[i][sp] = ld_nc_f4(gp + (size_t)sp * gs4);
                }
            }
            if (!mbar_wait(smem_u32(&accum_bar), (uint32_t)s & 1u, abort_flag)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // accumulator row = 4 * unit + gate; in pair mode rows [0, RA) belong to the even CTA's units and
            // rows [RA, 2 RA) to the odd CTA's: the partner's rows go to the partner's shared memory
            const int row = lq * 32 + lane;
            const int half = (pair && row >= RA) ? 1 : 0;
            const int lr = row - half * RA;
            const bool mine = !pair || half == rank;
            const bool row_ok = row < RT && lr < 4 * (mine ? nu : nu_partner);
            if (lq * 32 < (pair ? RT : 4 * nu)) {
                // the first four column chunks of 16 (all there are up to 32 sequences) are requested before
                // one wait; batches above 32 read their remaining chunks one at a time (registers)
                const int nchunk = (2 * B + 15) >> 4;
                {
                    float z[4][8];
                    // one issuer's accumulator after the other; hi and lo columns are added on the way
                    for (int wi = 0; wi < a.nissue; ++wi) {
                        uint32_t x[4][16];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            if (c < nchunk) tmem_ld16(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(wi * N + c * 16), x[c]);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            if (c < nchunk) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float zz = __uint_as_float(x[c][2 * i]) + __uint_as_float(x[c][2 * i + 1]);
                                    z[c][i] = wi ? z[c][i] + zz : zz;
                                }
                            }
                    }
                    if (row_ok) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if (c < nchunk) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const int b = c * 8 + i;
                                    if (b < B) {
                                        (mine ? zs : zsp)[b * zld + lr] = z[c][i];
                                    }
                                }
                            }
                        }
                    }
                }
#pragma unroll 1
                for (int c = 4; c < nchunk; ++c) {
                    uint32_t w[16];
                    tmem_ld16(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(c * 16), w);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    for (int wi = 1; wi < a.nissue; ++wi) {
                        uint32_t x[16];
                        tmem_ld16(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(wi * N + c * 16), x);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = __float_as_uint(__uint_as_float(w[i]) + __uint_as_float(x[i]));
                    }
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int b = c * 8 + i;
                            const float z = __uint_as_float(w[2 * i]) + __uint_as_float(w[2 * i + 1]);
                            if (b < B) {
                                (mine ? zs : zsp)[b * zld + lr] = z;
                            }
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            bar_sync(1, 128);
            if (pair) {
                // one bulk copy carries the partner's partial sums into its shared memory and completes on its
                // barrier; ours arrive the same way (bounded wait)
                if (ftid == 0) {
                    const uint32_t bytes = (uint32_t)(zld * B) * 4u;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_expect_tx(smem_u32(&partial_bar), bytes);
                    bulk_copy_to_cta(zs2_remote, smem_u32(zsp), bytes, partial_bar_remote);
                }
                if (!mbar_wait(smem_u32(&partial_bar), (uint32_t)s & 1u, abort_flag)) break;
            }
            __nv_bfloat16 *hp = hbuf_d + (size_t)(s & 1) * kTcPlaneRows * a.ldh;
            // one (unit, batch row) item: gates, c/h update, the new h as planes, outputs
            auto finish_item = [&](int p, int b, int u, const float4 &gsum) {
                const int j = u0 + u;
                float4 z4 = *reinterpret_cast<const float4 *>(zs + b * zld + 4 * u);
                if (pair) {
                    const float4 y4 = *reinterpret_cast<const float4 *>(zs2 + b * zld + 4 * u);
                    z4.x += y4.x; z4.y += y4.y; z4.z += y4.z; z4.w += y4.w;
                }
                const float gi = sigmoid_fast(z4.x + gsum.x);
                const float gf = sigmoid_fast(z4.y + gsum.y);
                const float gg = tanh_fast(z4.z + gsum.z);
                const float go = sigmoid_fast(z4.w + gsum.w);
                const float cn = fmaf(gf, c_s[p], gi * gg);
                const float hn = go * tanh_fast(cn);
                c_s[p] = cn;
                const __nv_bfloat16 hi = __float2bfloat16_rn(hn);
                const __nv_bfloat16 lo = __float2bfloat16_rn(hn - __bfloat162float(hi));
                hp[(size_t)(2 * b) * a.ldh + j] = hi;
                hp[(size_t)(2 * b + 1) * a.ldh + j] = lo;
                a.y[((size_t)t * B + b) * D * H + (size_t)d * H + j] = hn;
                if (a.xb_next) {
                    const size_t xi = ((size_t)t * B + b) * a.xb_ld + (size_t)d * H + j;
                    a.xb_next[xi] = hi;
                    a.xb_next[a.xb_plane + xi] = lo;
                }
                if (s == T - 1) {
                    if (a.hT) a.hT[((size_t)d * B + b) * H + j] = hn;
                    if (a.cT) a.cT[((size_t)d * B + b) * H + j] = cn;
                }
            };
            // consecutive threads, consecutive units; the first kPre items have their projection terms in registers
#pragma unroll
            for (int i = 0; i < kPre; ++i) {
                const int p = ftid + 128 * i;
                if (p < nuB) {
                    float4 gsum = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
                    for (int sp = 0; sp < kMaxSplit; ++sp)
                        if (sp < a.nsplit) { gsum.x += gpre[i][sp].x; gsum.y += gpre[i][sp].y; gsum.z += gpre[i][sp].z; gsum.w += gpre[i][sp].w; }
                    finish_item(p, pb[i], pu[i], gsum);
                }
            }
            for (int p = ftid + 128 * kPre; p < nuB; p += 128) {
                const int b = p / nu, u = p - b * nu;
                const float4 *gp = reinterpret_cast<const float4 *>(a.G + (((size_t)t * B + b) * D + d) * 4 * H + (size_t)(u0 + u) * 4);
                float4 gsum = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                for (int sp = 0; sp < a.nsplit; ++sp) {
                    const float4 g4 = __ldg(gp + (size_t)sp * gs4);
                    gsum.x += g4.x; gsum.y += g4.y; gsum.z += g4.z; gsum.w += g4.w;
                }
                finish_item(p, b, u, gsum);
            }
            bar_sync(1, 128);
            if (ftid == 0) {
                if ((int)blockIdx.x != a.withhold_cta) {
                    st_release_u32(flags_d + cta, a.stamp_base + (unsigned)s + 1u);
                }
                *pub = s + 2;
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
    if (pair) cluster_sync_all();               // no CTA leaves while its partner may still write into its shared memory
}

// rows x cols bf16 matrix, row stride ld elements; box = 64 columns x box_rows, 128-byte swizzle, zero fill
bool encode_2d(void *map, const void *base, long long rows, int cols, int ld, int box_rows)
{
    return encode_tmap_bf16_2d(map, base, rows, cols, ld, box_rows);
}

}  // namespace

static_assert(sizeof(CUtensorMap) == 128, "tensor map size");

size_t recur_tc_smem_bytes(int RA, int nkb, int N, int stages, int kbs, int upc, int B, int pair)
{
    // pair mode: tiles of 2 RA rows, half of the K blocks (rounded up), and a second block of partial sums
    const int RT = pair ? 2 * RA : RA, nkb_alloc = pair ? (nkb + 1) / 2 : nkb;
    // the last weight tile is read as 128 rows: at least (128 - RT) * 128 bytes must follow it
    const size_t scratch = (size_t)(4 * upc * B) * (pair ? 3 : 1) + (size_t)((upc * B + 3) & ~3);
    const size_t after = (size_t)stages * kbs * N * 128 + scratch * 4 + 16;
    const size_t need = (size_t)(128 - RT) * 128;
    return 1024 + (size_t)nkb_alloc * RT * 128 + (after > need ? after : need);
}

// Ring shape for one launch: stages of up to four K blocks (one mbarrier round trip per stage instead of per
// block); a ring that holds the whole operand if one fits, else as many stages as fit, at least two.
bool recur_tc_plan(int RA, int nkb, int N, int upc, int B, size_t max_smem, int pair, int *kbs_out, int *stages_out)
{
    const int nkb_cta = pair ? (nkb + 1) / 2 : nkb;
    if (pair && (2 * RA > 128 || nkb < 2)) return false;
    // first choice: a ring that holds a whole step's operand (all copies of a step are then issued together),
    // in as few stages as possible
    for (int kbs = nkb_cta < 4 ? nkb_cta : 4; kbs >= 1 && nkb_cta <= 32; --kbs) {
        const int st = (nkb_cta + kbs - 1) / kbs;
        if (st <= kMaxStages && recur_tc_smem_bytes(RA, nkb, N, st, kbs, upc, B, pair) <= max_smem) {
            *kbs_out = kbs;
            *stages_out = st;
            return true;
        }
    }
    for (int kbs = nkb_cta < 4 ? nkb_cta : 4; kbs >= 1; --kbs) {
        const int groups = (nkb_cta + kbs - 1) / kbs;
        for (int st = groups < kMaxStages ? groups : kMaxStages; st >= (groups > 1 ? 2 : 1); --st) {
            if (recur_tc_smem_bytes(RA, nkb, N, st, kbs, upc, B, pair) <= max_smem) {
                *kbs_out = kbs;
                *stages_out = st;
                return true;
            }
        }
    }
    return false;
}

bool recur_tc_encode_weights(void *map, const void *w, long long rows, int ld, int RA)
{
    return encode_2d(map, w, rows, ld, ld, RA);
}
bool recur_tc_encode_planes(void *map, const void *hbuf, int D, int H, int ldh, int B)
{
    // a box holds the 2B plane rows rounded up to a swizzle group of 8, not the MMA's N (a multiple of 16)
    return encode_2d(map, hbuf, (long long)D * 2 * kTcPlaneRows, H, ldh, (2 * B + 7) & ~7);
}

cudaError_t recur_tc_prepare(int max_smem)
{
    return cudaFuncSetAttribute(recur_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

// Can `grid` CTAs of this kernel be co-resident as clusters of two (pair mode needs every pair on one GPC)?
bool recur_tc_pair_supported(int grid, size_t smem)
{
    if (grid < 2 || (grid & 1)) return false;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, (const void *)recur_tc_kernel, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return clusters * 2 >= grid;
}

cudaError_t launch_recur_tc(const void *tmap_w, const void *tmap_h, const RecurTcArgs &a, size_t smem, cudaStream_t st)
{
    CUtensorMap mw, mh;
    memcpy(&mw, tmap_w, sizeof mw);
    memcpy(&mh, tmap_h, sizeof mh);
    RecurTcArgs copy = a;
    void *params[] = {&mw, &mh, &copy};
    const int grid = a.ncta_dir * (a.ndirs ? a.ndirs : a.D);
    if (!a.pair)
        return cudaLaunchCooperativeKernel((const void *)recur_tc_kernel, dim3(grid), dim3(kThreads), params, smem, st);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelExC(&cfg, (const void *)recur_tc_kernel, params);
}

}  // namespace lstm
