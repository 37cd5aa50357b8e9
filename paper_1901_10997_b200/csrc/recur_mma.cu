// Register-resident recurrent kernel for bf16 weights: the serial half of the LSTM forward pass
// (paper, Section 4, cell equations with zero hidden layers per gate)
//     z = G[t] + Wh h_{t-1};  i,f,o = sigmoid(z_i,z_f,z_o), g = tanh(z_g);  c_t = f c_{t-1} + i g;
//     h_t = o tanh(c_t)
// with G[t] the input projection (bias included) computed for all timesteps beforehand.
//
// Design.  One cooperative launch runs all T steps of one layer (both directions side by side on
// disjoint CTA groups).  A CTA owns a contiguous range of hidden units (all four gate rows of a unit)
// and keeps its slice of Wh in the REGISTER FILE for the whole sequence: the slice is cut into
// 16 x 16 tiles stored in the operand-A fragment layout of mma.sync.m16n8k16, warp w holding the tiles
// of its own column range for every row tile (tiles that do not fit the register budget sit in shared
// memory in the same layout).  A step therefore reads no weight from shared memory or L2 at all: each
// warp polls only the h values of its own column range, splits them into bf16 hi + lo parts (batch row
// b occupies columns 2b and 2b+1 of the 8-wide B operand), issues MT x NKW tensor-core instructions and
// leaves per-warp partial sums in shared memory; after one CTA barrier warp w finishes unit w: its lanes
// add the partials and the projection term of a (batch row, gate), apply the gate function, and one lane
// per batch row updates c and h and publishes h.  tcgen05.mma cannot take its A operand from registers and re-reading
// it from shared memory every step is exactly the cost this kernel removes, so the warp-level mma is
// the right instruction here.
//
// Exchange of h_t: every value is published as one 64-bit word {step stamp, value}; consumers poll the
// words themselves, so a step costs one L2 round trip after the last producer's store and there is no
// grid barrier.  A warp starts to poll for step s+1 right after it has published its unit of step s, so
// the CTAs run in near lock-step and a poll seldom has to be repeated (warps that spin on words that are
// not there yet delay the very stores they wait for).  Inside a CTA the only synchronisation per step
// is one named barrier between the partial sums and their consumers (consecutive steps alternate
// between two barriers and two partial-sum buffers).  Every wait on another CTA is bounded: when it
// expires the CTA records a timeout status, stops waiting for the rest of the launch and runs to the end.
#include "common.cuh"
#include "device_util.cuh"
#include "recur_parts.cuh"

#include <algorithm>

namespace lstm {
namespace {





constexpr int kPoll = 4;      // exchange words a lane keeps in flight per polling round
constexpr int kMaxSplit = 4;  // split-K planes of the projection output (the projection plans at most 4)
constexpr int kMaxPairs = 12;  // pairs of exchange words per lane in a staged pass: 4 rows x up to 192 columns
constexpr int kChunk = 4;     // batch rows per pass: hi and lo parts fill the 8 columns of the B operand

// MT: 16-row tiles per CTA (4 gate rows x units, padded); NKR: 16-column tiles per warp held in
// registers; NW: warps per CTA.
// STAGED: the pass over several batch rows that lands the exchange words in shared memory (cp.async); kept
// out of the single-row instantiation, whose registers are all spoken for.
// ONE: a single sequence (B = 1): the batch-row arithmetic folds away at compile time.
// POLL3: a lane polls three words per round instead of four (single sequence, at most 96 columns per warp).
// PROBE: the measurement build of the single-sequence variants, which honours a.probe (parts of a step left
// out); in every other instantiation the probe tests fold away, so the production step carries none of them.
// FUSE: single short sequence (T <= kFuseMaxT): the CTA computes its own rows of the layer's input projection
// G = X Wx^T + b in the prologue (Wx fragments streamed once from global memory, X split into bf16 hi + lo on
// the fly) and keeps them in shared memory, instead of reading a G computed by a separate launch.
template <int MT, int NKR, int NW, bool STAGED, bool ONE, bool POLL3, bool PROBE = false, bool FUSE = false>
__global__ void __launch_bounds__(NW * 32, 1) recur_mma_kernel(const RecurMmaArgs a)
{
    const int probe = PROBE ? a.probe : 0;
    constexpr int NT = NW * 32;
    constexpr int RP = MT * 16 + 8;          // row pitch of the partial sums: conflict-free writes
    constexpr int WS = 4 * RP + 4;           // pitch between warps: the readers of one row spread over the banks
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int abort_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int H = a.H, B = ONE ? 1 : a.B, T = a.T, D = a.D;
    const int d = a.dir0 + blockIdx.x / a.ncta_dir;
    const int cta = blockIdx.x % a.ncta_dir;
    int u0, nu;
    unit_range(H, a.ncta_dir, cta, u0, nu);
    const int upc = (H + a.ncta_dir - 1) / a.ncta_dir;
    const int nks = a.nkw_smem, nkw = NKR + nks;
    const int kspan = nkw * 16, kbase = warp * kspan;

    // ---- shared-memory carve-up
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem);                  // [NW][nkw][8][16]
    float *red = reinterpret_cast<float *>(smem + (size_t)NW * nkw * 256);        // [2][NW][WS] as [4][RP] + pad
    float *c_s = red + 2 * NW * WS;                                           // [upc][B]
    uint4 *As = reinterpret_cast<uint4 *>(c_s + ((upc * B + 3) & ~3));            // [NW][nks][MT][32]
    // landing area of the exchange words of a pass over several batch rows: [NW][kChunk][kspan]
    unsigned long long *stage = reinterpret_cast<unsigned long long *>(As + (size_t)NW * nks * MT * 32);
    // fused projection: this CTA's rows of G for every timestep, [kFuseMaxT][GP], behind everything else
    constexpr int GP = MT * 16 + 1;
    float *G_s = nullptr;
    LSTM_CHECK_SMEM_END(reinterpret_cast<unsigned char *>(stage) - smem + (STAGED ? (size_t)NW * kChunk * kspan * 8 : 0), a.status);
    if (FUSE) LSTM_CHECK_SMEM_END((size_t)a.gs_off + (size_t)kFuseMaxT * GP * 4, a.status);
    if (FUSE) LSTM_CHECK_SMEM_END((size_t)NW * 24 * GP * 4, a.status);

    const uint4 *wsrc = a.wfrag[d] + ((size_t)(cta * NW + warp) * nkw) * MT * 32 + lane;
    if (FUSE) {
        // ---- the CTA's rows of the input projection.  Both weight streams are requested into L2 at once, so that
        // they leave HBM side by side; the registers the recurrent fragments will live in are free until the end.
        for (int i = lane; i < nkw * MT * 4; i += 32)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(wsrc - lane) + (size_t)i * 128));
        G_s = fused_projection<MT, NW>(smem, (size_t)a.gs_off, a.X, a.xfrag[d], a.bias, a.nkw_x, a.in_l, T, H, d, cta, u0, nu, tid);
    }
    // ---- residency: this warp's tiles, registers first, the rest in shared memory
    uint4 areg[NKR][MT];
#pragma unroll
    for (int i = 0; i < NKR; ++i)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) areg[i][mt] = __ldg(wsrc + (size_t)(i * MT + mt) * 32);
    uint4 *As_w = As + (size_t)warp * nks * MT * 32 + lane;
    for (int i = 0; i < nks * MT; ++i) As_w[(size_t)i * 32] = __ldg(wsrc + (size_t)(NKR * MT + i) * 32);

    for (int i = tid; i < NW * nkw * 64; i += NT) reinterpret_cast<unsigned *>(Bs)[i] = 0u;
    for (int i = tid; i < 2 * NW * WS; i += NT) red[i] = 0.0f;
    for (int i = tid; i < nu * B; i += NT) {
        const int u = i / B, b = i - u * B;
        c_s[u * B + b] = a.c0 ? a.c0[((size_t)d * B + b) * H + u0 + u] : 0.0f;
    }
    if (tid == 0) abort_s = 0;
    __syncthreads();
    volatile int *abort_v = &abort_s;

    const int nchunk = (B + kChunk - 1) / kChunk;
    unsigned long long *xch_d = a.xch + (size_t)d * 2 * B * H;
    __nv_bfloat16 *Bw = Bs + (size_t)warp * nkw * 128;
    const unsigned *Bw32 = reinterpret_cast<const unsigned *>(Bw);

    // Finishing role: warp w finishes unit w of this CTA.  With nbe = 1, 2 or 4 batch rows per pass the
    // 32 lanes split into nbe * 4 (batch row, gate) groups of P = 8 / nbe lanes; the lanes of a group
    // share the sum over the warps' partial results and lane 0 of the group applies the gate function.
    const int nbe = B >= 3 ? 4 : B;                 // batch rows a pass is laid out for
    const int P = 8 / nbe;
    const int fpart = lane % P, fgrp = lane / P;    // fgrp = fb * 4 + fq
    const int fb = fgrp >> 2, fq = fgrp & 3;
    const bool fin_warp = warp < nu;
    // gate function of this lane's gate (fq == 2: the cell candidate, tanh; else the logistic function)
    const float act_k = (fq == 2 ? -2.0f : -1.0f) * 1.4426950408889634f, act_sc = fq == 2 ? 2.0f : 1.0f, act_of = fq == 2 ? -1.0f : 0.0f;
    const int frow = warp * 4 + fq;

    // Warps whose column range lies beyond H have nothing to poll and finish no unit: they leave now
    // (their partial sums stay zero).  The per-step barrier counts the remaining warps only.
    const int n_active = (H + kspan - 1) / kspan;
    const int nbar = 32 * max(n_active, nu);
    if (warp * 32 >= nbar) return;

    // Projection term of this lane's (batch row, gate) of unit `warp` at processing step s, chunk ci: one
    // value per split-K plane, summed only where it is used, so that the loads stay in flight meanwhile.
    struct GTerm { float v[kMaxSplit]; };
    auto load_g = [&](int s, int ci) -> GTerm {
        GTerm r;
#pragma unroll
        for (int sp = 0; sp < kMaxSplit; ++sp) r.v[sp] = 0.0f;
        const int b = ci * kChunk + fb;
        if (FUSE) {
            if (fin_warp && fpart == 0 && s < T) r.v[0] = G_s[(size_t)(d ? (T - 1 - s) : s) * GP + warp * 4 + fq];
        } else if (fin_warp && fpart == 0 && s < T && b < B) {
            const int t = d ? (T - 1 - s) : s;
            const float *gp = a.G + (((size_t)t * B + b) * D + d) * 4 * H + (size_t)(u0 + warp) * 4 + fq;
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp)
                if (sp < a.nsplit) r.v[sp] = ld_nc_early(gp + (size_t)sp * a.g_split_stride);
        }
        return r;
    };
    // Exchange word idx of a pass over nb rows is element idx of the warp's [nb][kspan] block: offset
    // in the exchange buffer, offset in the staged operand, and whether the column exists.
    auto word_offsets = [&](int idx, int &so, int &dof) -> bool {
        int b = 0, kk = idx;
        if (B > 1) { b = idx / kspan; kk = idx - b * kspan; }
        so = b * H + kbase + kk;
        dof = ((kk >> 4) * 8 + 2 * b) * 16 + (kk & 15);
        return kbase + kk < H;
    };

    int it = 0;
    // two steps per loop body where registers allow it: the buffer parities become constants
#pragma unroll(ONE && MT * NKR <= 12 ? 2 : 1)
    for (int s = 0; s < T; ++s) {
        const int t = d ? (T - 1 - s) : s;
#pragma unroll 1
        for (int ci = 0; ci < nchunk; ++ci, ++it) {
            const int b0 = ci * kChunk;
            const int nb = min(kChunk, B - b0);
            // projection term of this pass: requested now, needed only after the products below
            const GTerm g_cur = load_g(s, ci);

            // ---- this warp's columns of h_{t-1}, rows b0 .. b0+nb-1, as bf16 hi/lo parts in operand-B order
            const int nwords = nb * kspan;
            if (s == 0) {
                for (int idx = lane; idx < nwords; idx += 32) {
                    int so, dof;
                    if (word_offsets(idx, so, dof)) {
                        const float v = a.h0 ? a.h0[((size_t)d * B + b0) * H + so] : 0.0f;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                        Bw[dof] = hi;
                        Bw[dof + 16] = __float2bfloat16_rn(v - __bfloat162float(hi));
                    }
                }
            } else if (probe & kProbeNoExchange) {
                // measurement only: no wait for the other CTAs, the operand keeps whatever it holds
            } else if (STAGED) {
                // Several batch rows: too many words per lane to hold in registers at once, and polling
                // them in rounds would cost one L2 round trip per round.  All words of the pass are
                // copied to shared memory asynchronously in one go (pairs of words, 16 bytes); pairs whose
                // stamps are not there yet are requested again.
                const unsigned want = a.stamp_base + (unsigned)s;
                const unsigned long long *src = xch_d + ((size_t)((s - 1) & 1) * B + b0) * H + kbase;
                unsigned long long *stg = stage + (size_t)warp * kChunk * kspan;
                unsigned todo = 0;                                     // bit j: pair 2*lane + 64*j still missing
#pragma unroll
                for (int j = 0; j < kMaxPairs; ++j) {
                    const int idx = 2 * lane + 64 * j;
                    if (idx < nwords) {
                        const int b = (idx >= kspan) + (idx >= 2 * kspan) + (idx >= 3 * kspan), kk = idx - b * kspan;
                        if (kbase + kk < H) todo |= 1u << j;
                    }
                }
                if (*abort_v) todo = 0;
                long long t_start = 0;
                int rounds = 0;
                while (__any_sync(0xffffffffu, todo != 0)) {
#pragma unroll
                    for (int j = 0; j < kMaxPairs; ++j)
                        if (todo & (1u << j)) {
                            const int idx = 2 * lane + 64 * j;
                            const int b = (idx >= kspan) + (idx >= 2 * kspan) + (idx >= 3 * kspan), kk = idx - b * kspan;
                            cp_async_16(stg + idx, src + (size_t)b * H + kk);
                        }
                    cp_async_wait_all();
#pragma unroll
                    for (int j = 0; j < kMaxPairs; ++j)
                        if (todo & (1u << j)) {
                            const int idx = 2 * lane + 64 * j;
                            const ulonglong2 w = *reinterpret_cast<const ulonglong2 *>(stg + idx);
                            if ((unsigned)(w.x >> 32) == want && (unsigned)(w.y >> 32) == want) {
                                const int b = (idx >= kspan) + (idx >= 2 * kspan) + (idx >= 3 * kspan), kk = idx - b * kspan;
                                const float v0 = __uint_as_float((unsigned)w.x), v1 = __uint_as_float((unsigned)w.y);
                                const __nv_bfloat162 hi = __floats2bfloat162_rn(v0, v1);
                                const __nv_bfloat162 lo = __floats2bfloat162_rn(v0 - __low2float(hi), v1 - __high2float(hi));
                                const int dof = ((kk >> 4) * 8 + 2 * b) * 16 + (kk & 15);      // kk even: one 32-bit store
                                *reinterpret_cast<__nv_bfloat162 *>(Bw + dof) = hi;
                                *reinterpret_cast<__nv_bfloat162 *>(Bw + dof + 16) = lo;
                                todo &= ~(1u << j);
                            }
                        }
                    if (todo && ((++rounds & 15) == 0)) {
                        const long long now = clock64();
                        if (t_start == 0) t_start = now;
                        if (*abort_v) todo = 0;
                        else if (now - t_start > a.spin_limit || ld_volatile_s32(a.status) != kStatusOk) {
                            *abort_v = 1;
                            atomicExch(a.status, kStatusTimeout);
                            todo = 0;
                        }
                    }
                }
            } else {
                const unsigned want = a.stamp_base + (unsigned)s;            // stamp of step s-1
                const unsigned long long *src = xch_d + ((size_t)((s - 1) & 1) * B + b0) * H;
                long long t_start = 0;
                constexpr int KP = POLL3 ? 3 : kPoll;
                for (int base = 0; base < nwords; base += 32 * KP) {
                    unsigned pending = 0;
                    int soff[KP], doff[KP];
#pragma unroll
                    for (int i = 0; i < KP; ++i) {
                        const int idx = base + lane + 32 * i;
                        if (word_offsets(idx, soff[i], doff[i]) && idx < nwords) pending |= 1u << i;
                    }
                    if (*abort_v) pending = 0;
                    int rounds = 0;
                    while (pending) {
                        unsigned long long w[KP];
#pragma unroll
                        for (int i = 0; i < KP; ++i)
                            if (pending & (1u << i)) w[i] = ld_relaxed_u64(src + soff[i]);
#pragma unroll
                        for (int i = 0; i < KP; ++i)
                            if ((pending & (1u << i)) && (unsigned)(w[i] >> 32) == want) {
                                const float v = __uint_as_float((unsigned)w[i]);
                                const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                                if (LSTM_CHECK_INDEX(doff[i] + 16, nkw * 128, a.status)) {
                                    Bw[doff[i]] = hi;
                                    Bw[doff[i] + 16] = __float2bfloat16_rn(v - __bfloat162float(hi));
                                }
                                pending &= ~(1u << i);
                            }
                        if (pending && ((++rounds & 63) == 0)) {
                            const long long now = clock64();
                            if (t_start == 0) t_start = now;
                            if (*abort_v) pending = 0;
                            else if (now - t_start > a.spin_limit || ld_volatile_s32(a.status) != kStatusOk) {
                                *abort_v = 1;
                                atomicExch(a.status, kStatusTimeout);
                                pending = 0;
                            }
                        }
                    }
                }
            }
            __syncwarp();

            // ---- partial products of this warp's columns: registers first, then the shared-memory tiles
            float acc[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
            if (!(probe & kProbeNoProducts)) {
#pragma unroll
                for (int i = 0; i < NKR; ++i) {
                    const unsigned bv0 = Bw32[i * 64 + g * 8 + tig];
                    const unsigned bv1 = Bw32[i * 64 + g * 8 + tig + 4];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], areg[i][mt], bv0, bv1);
                }
                for (int i = 0; i < nks; ++i) {
                    const unsigned bv0 = Bw32[(NKR + i) * 64 + g * 8 + tig];
                    const unsigned bv1 = Bw32[(NKR + i) * 64 + g * 8 + tig + 4];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], As_w[(size_t)(i * MT + mt) * 32], bv0, bv1);
                }
            }
            // accumulator columns 2*tig and 2*tig+1 are the hi and lo parts of batch row tig
            float *rw = red + (size_t)((it & 1) * NW + warp) * WS + tig * RP + g;
            if (LSTM_CHECK_INDEX((rw - red) + (MT - 1) * 16 + 8, 2 * NW * WS, a.status)) {
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    rw[mt * 16] = acc[mt][0] + acc[mt][1];
                    rw[mt * 16 + 8] = acc[mt][2] + acc[mt][3];
                }
            }

            // ---- all partial sums of this pass are in place (two barriers and two buffers alternate)
            bar_sync(1 + (it & 1), nbar);

            if (fin_warp && (probe & kProbeNoGates)) {
                // measurement only: the exchange without the reduction, the gate functions and the outputs
                if (fq == 0 && fpart == 0 && fb < nb && (int)blockIdx.x != a.withhold_cta)
                    st_relaxed_u64(xch_d + ((size_t)(s & 1) * B + b0 + fb) * H + u0 + warp,
                                   ((unsigned long long)(a.stamp_base + (unsigned)s + 1u) << 32) | 0x3e800000ull);
            } else if (fin_warp) {
                float z = 0.0f;
                if (fb < nb) {
                    const float *rp = red + (size_t)((it & 1) * NW) * WS + fb * RP + frow;
                    for (int w = fpart; w < NW; w += P) z += rp[(size_t)w * WS];
                }
                for (int o = P >> 1; o >= 1; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                z += (g_cur.v[0] + g_cur.v[1]) + (g_cur.v[2] + g_cur.v[3]);
                const float act = gate_fast(z, act_k, act_sc, act_of);
                const int qb = fb * 4 * P;                 // lane of gate i of this batch row
                const float vi = __shfl_sync(0xffffffffu, act, qb);
                const float vf = __shfl_sync(0xffffffffu, act, qb + P);
                const float vg = __shfl_sync(0xffffffffu, act, qb + 2 * P);
                const float vo = __shfl_sync(0xffffffffu, act, qb + 3 * P);
                if (fq == 0 && fpart == 0 && fb < nb) {
                    const int b = b0 + fb, j = u0 + warp;
                    const float cn = fmaf(vf, c_s[warp * B + b], vi * vg);
                    const float hn = vo * tanh_fast(cn);
                    if ((int)blockIdx.x != a.withhold_cta)
                    st_relaxed_u64(xch_d + ((size_t)(s & 1) * B + b) * H + j,
                                   ((unsigned long long)(a.stamp_base + (unsigned)s + 1u) << 32) |
                                       (unsigned long long)__float_as_uint(hn));
                    c_s[warp * B + b] = cn;
                    a.y[((size_t)t * B + b) * D * H + (size_t)d * H + j] = hn;
                    if (a.xb_next) {
                        const size_t xi = ((size_t)t * B + b) * a.xb_ld + (size_t)d * H + j;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(hn);
                        a.xb_next[xi] = hi;
                        a.xb_next[a.xb_plane + xi] = __float2bfloat16_rn(hn - __bfloat162float(hi));
                    }
                    if (s == T - 1) {
                        if (a.hT) a.hT[((size_t)d * B + b) * H + j] = hn;
                        if (a.cT) a.cT[((size_t)d * B + b) * H + j] = cn;
                    }
                }
            }
            // Warps that finish no unit must not start to poll before this CTA has issued its own stores:
            // their loads would sit in front of those stores on the way to L2.
            if (nchunk == 1 && nbar > 32 * nu) {
                if (fin_warp) bar_arrive(3 + (it & 1), nbar);
                else bar_sync(3 + (it & 1), nbar);
            }
        }
    }
}

typedef void (*KernelFn)(const RecurMmaArgs);

template <int MT, int NW, bool STAGED, bool ONE, bool POLL3, bool PROBE, bool FUSE>
KernelFn pick_nkr(int nkr)
{
    switch (nkr) {
        case 2: return recur_mma_kernel<MT, 2, NW, STAGED, ONE, POLL3, PROBE, FUSE>;
        case 4: return recur_mma_kernel<MT, 4, NW, STAGED, ONE, POLL3, PROBE, FUSE>;
        case 6: return recur_mma_kernel<MT, 6, NW, STAGED, ONE, POLL3, PROBE, FUSE>;
        case 8: return recur_mma_kernel<MT, 8, NW, STAGED, ONE, (POLL3 && false), PROBE, FUSE>;     // 128 columns per warp: four words
        default: return nullptr;
    }
}
template <int NW, bool STAGED, bool ONE, bool POLL3, bool PROBE = false, bool FUSE = false>
KernelFn pick_mt(int mt, int nkr)
{
    switch (mt) {
        case 1: return pick_nkr<1, NW, STAGED, ONE, POLL3, PROBE, FUSE>(nkr);
        case 2: return pick_nkr<2, NW, STAGED, ONE, POLL3, PROBE, FUSE>(nkr);
        case 3: return pick_nkr<3, NW, STAGED, ONE, POLL3, PROBE, FUSE>(nkr);
        case 4: return pick_nkr<4, NW, STAGED, ONE, POLL3, PROBE, FUSE>(nkr);
        default: return nullptr;
    }
}
// variant 0: several rows polled from registers, 1: several rows staged in shared memory, 2: one sequence,
// 3: one sequence with at most 96 columns per warp (three polled words per lane); 4, 5: the measurement
// builds of 2 and 3; 6, 7: 2 and 3 with the input projection of a short sequence fused into the prologue
KernelFn pick(int mt, int nkr, int nw, int variant)
{
    if (!recur_mma_shape_ok(mt, nkr, nw)) return nullptr;
    if (variant == 4) return nw == 8 ? pick_mt<8, false, true, false, true>(mt, nkr) : pick_mt<16, false, true, false, true>(mt, nkr);
    if (variant == 5) return nw == 8 ? pick_mt<8, false, true, true, true>(mt, nkr) : pick_mt<16, false, true, true, true>(mt, nkr);
    if (variant == 6) return nw == 8 ? pick_mt<8, false, true, false, false, true>(mt, nkr) : pick_mt<16, false, true, false, false, true>(mt, nkr);
    if (variant == 7) return nw == 8 ? pick_mt<8, false, true, true, false, true>(mt, nkr) : pick_mt<16, false, true, true, false, true>(mt, nkr);
    if (variant == 1) return nw == 8 ? pick_mt<8, true, false, false>(mt, nkr) : pick_mt<16, true, false, false>(mt, nkr);
    if (variant == 2) return nw == 8 ? pick_mt<8, false, true, false>(mt, nkr) : pick_mt<16, false, true, false>(mt, nkr);
    if (variant == 3) return nw == 8 ? pick_mt<8, false, true, true>(mt, nkr) : pick_mt<16, false, true, true>(mt, nkr);
    return nw == 8 ? pick_mt<8, false, false, false>(mt, nkr) : pick_mt<16, false, false, false>(mt, nkr);
}

}  // namespace

bool recur_mma_shape_ok(int mt, int nkr, int nw)
{
    if (mt < 1 || mt > 4 || (nkr != 2 && nkr != 4 && nkr != 6 && nkr != 8)) return false;
    if (nw == 16) return mt * nkr <= kMmaTileCap16;
    if (nw == 8) return mt * nkr <= kMmaTileCap8;
    return false;
}

// fused projection: the partial products of all warps (24 timesteps x rows each) lie over the kernel's other
// shared memory, the finished rows of G behind whichever is larger
size_t recur_mma_fuse_gs_offset(int mt, int nkr, int nw, int nkw_smem, int upc)
{
    const size_t normal = recur_mma_smem_bytes(mt, nkr, nw, nkw_smem, upc, 1, false, false);
    const size_t partial = (size_t)nw * 24 * (mt * 16 + 1) * 4;
    return (std::max(normal, partial) + 15) & ~(size_t)15;
}

size_t recur_mma_smem_bytes(int mt, int nkr, int nw, int nkw_smem, int upc, int B, bool staged, bool fused)
{
    const int nkw = nkr + nkw_smem;
    if (fused) return recur_mma_fuse_gs_offset(mt, nkr, nw, nkw_smem, upc) + (size_t)kFuseMaxT * (mt * 16 + 1) * 4;
    return (staged ? (size_t)nw * kChunk * nkw * 16 * 8 : 0) + (size_t)nw * nkw * 256 + (size_t)2 * nw * (4 * (mt * 16 + 8) + 4) * 4 +
           (size_t)((upc * B + 3) & ~3) * 4 + (size_t)nw * nkw_smem * mt * 512;
}

cudaError_t recur_mma_prepare(int mt, int nkr, int nw, int max_smem)
{
    for (int variant = 0; variant < 8; ++variant) {
        KernelFn fn = pick(mt, nkr, nw, variant);
        if (!fn) return cudaErrorInvalidValue;
        const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_recur_mma(const RecurMmaArgs &a, int mt, int nkr, int nw, size_t smem, cudaStream_t st)
{
    int variant = a.staged ? 1 : a.B != 1 ? 0 : (nkr + a.nkw_smem) * 16 <= 96 ? 3 : 2;
    if (a.probe) {
        if (variant < 2 || a.fuse) return cudaErrorInvalidValue;      // probe modes exist for the plain single-sequence variants only
        variant += 2;
    }
    if (a.fuse) {
        if (variant < 2 || a.T > kFuseMaxT || !a.xfrag[0] || !a.X) return cudaErrorInvalidValue;
        variant += 4;
    }
    KernelFn fn = pick(mt, nkr, nw, variant);
    if (!fn) return cudaErrorInvalidValue;
    RecurMmaArgs copy = a;
    void *params[] = {&copy};
    return cudaLaunchCooperativeKernel((const void *)fn, dim3(a.ncta_dir * (a.ndirs ? a.ndirs : a.D)), dim3(nw * 32), params, smem, st);
}

}  // namespace lstm
