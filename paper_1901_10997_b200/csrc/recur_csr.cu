// Register-resident sparse recurrent kernel for pruned bf16 weights: the serial half of the LSTM forward
// pass (paper, Section 4, cell equations with zero hidden layers per gate) over the SURVIVING weights only
// (Section 4, mask-based pruning: W (x) Msk; here the zeros are never stored or multiplied):
//     z = G[t] + CSR(Wh) h_{t-1};  i,f,o = sigmoid(z_i,z_f,z_o), g = tanh(z_g);  c_t = f c_{t-1} + i g;
//     h_t = o tanh(c_t)
//
// Design.  The structure is the dense register-resident kernel's: one cooperative launch runs all T steps of
// a layer, a CTA owns a contiguous range of hidden units (all four gate rows of each), warp w of the CTA owns
// a column range of h and polls only those stamped words, and after one CTA barrier warp w finishes unit w.
// What differs is the product.  At 10 % density a CTA's slice is about 6600 weights, 13 per thread: it lives
// in REGISTERS for the whole sequence.  Inside a warp every lane owns up to two of the CTA's gate rows; its
// register list holds the surviving weights of those rows inside the warp's column range, one 32-bit word
// each {bf16 value | second-row flag | column}.  A step is then: poll the warp's words into a small fp32
// staging row in shared memory, run the register list (one shared-memory gather and two fused multiply-adds
// per entry, h in full fp32: no bf16 rounding of activations at all), write the lane's two partial sums.
// The lists are laid out at create time: rows are dealt to lanes longest-first so the lists have nearly equal
// length, and the entries of the 32 lanes are ordered so that the gathers of one slot fall into different
// shared-memory banks wherever the pattern allows it.
// Every wait on another CTA is bounded: when it expires the CTA records a timeout status, stops waiting for
// the rest of the launch and runs to the end.
#include "common.cuh"
#include "device_util.cuh"
#include "recur_parts.cuh"

#include <algorithm>

namespace lstm {
namespace {

constexpr int kChunk = 4;      // batch rows per pass
constexpr int kMaxSplit = 4;   // split-K planes of the projection output

// E: entry slots per lane; NW: warps per CTA; ONE: a single sequence (B = 1); PROBE: measurement build;
// FUSE: the CTA computes its own rows of the layer's input projection in the prologue (single short sequence),
// on the tensor cores over a dense copy of Wx, and reads the projection terms from shared memory afterwards.
template <int E, int NW, bool ONE, bool PROBE, bool FUSE = false>
__global__ void __launch_bounds__(NW * 32, 1) recur_csr_kernel(const RecurCsrArgs a)
{
    constexpr int NT = NW * 32;
    constexpr int NB = ONE ? 1 : kChunk;
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int abort_s;
    const int probe = PROBE ? a.probe : 0;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = a.H, B = ONE ? 1 : a.B, T = a.T, D = a.D;
    const int d = a.dir0 + blockIdx.x / a.ncta_dir;
    const int cta = blockIdx.x % a.ncta_dir;
    int u0, nu;
    unit_range(H, a.ncta_dir, cta, u0, nu);
    const int upc = (H + a.ncta_dir - 1) / a.ncta_dir;
    const int kspan = a.kspan, kbase = warp * kspan;
    const int RP = red_row_pitch(a.mt), WS = red_warp_pitch(a.mt);

    // ---- shared-memory carve-up.  The staging rows come first and every warp's block of them starts at a
    // multiple of a power of two >= its size, so that a gather address is (block offset | entry offset): one
    // logic instruction, no add.
    const int hstride = a.hs_stride;                             // floats per warp block
    float *hs = reinterpret_cast<float *>(smem);                 // [NW][hstride]: NB rows of kspan staged h values
    float *red = hs + (size_t)NW * hstride;                      // [2][NW][WS]
    float *c_s = red + 2 * NW * WS;                              // [upc][B]
    LSTM_CHECK_SMEM_END((size_t)(reinterpret_cast<unsigned char *>(c_s + ((upc * B + 3) & ~3)) - smem), a.status);

    // ---- the CTA's rows of the input projection (before anything else lives in shared memory or registers)
    const float *G_s = nullptr;
    const int GP = a.mt * 16 + 1;
    if (FUSE) {
        LSTM_CHECK_SMEM_END((size_t)a.gs_off + (size_t)kFuseMaxT * GP * 4, a.status);
        LSTM_CHECK_SMEM_END((size_t)NW * 24 * GP * 4, a.status);
        switch (a.mt) {
            case 1: G_s = fused_projection<1, NW>(smem, (size_t)a.gs_off, a.X, a.xfrag[d], a.bias, a.nkw_x, a.in_l, T, H, d, cta, u0, nu, tid); break;
            case 2: G_s = fused_projection<2, NW>(smem, (size_t)a.gs_off, a.X, a.xfrag[d], a.bias, a.nkw_x, a.in_l, T, H, d, cta, u0, nu, tid); break;
            case 3: G_s = fused_projection<3, NW>(smem, (size_t)a.gs_off, a.X, a.xfrag[d], a.bias, a.nkw_x, a.in_l, T, H, d, cta, u0, nu, tid); break;
            default: G_s = fused_projection<4, NW>(smem, (size_t)a.gs_off, a.X, a.xfrag[d], a.bias, a.nkw_x, a.in_l, T, H, d, cta, u0, nu, tid); break;
        }
    }

    // ---- residency: this lane's entry list and its rows
    unsigned ent[E];
    {
        const unsigned *esrc = a.ent[d] + ((size_t)(cta * NW + warp) * E) * 32 + lane;
#pragma unroll
        for (int e = 0; e < E; ++e) ent[e] = __ldg(esrc + (size_t)e * 32);
    }
    const unsigned rw = __ldg(a.rows[d] + (size_t)(cta * NW + warp) * 32 + lane);
    const int rowA = rw & 0xff, rowB = (rw >> 8) & 0xff;

    for (int i = tid; i < NW * hstride; i += NT) hs[i] = 0.0f;
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
    float *hsw = hs + (size_t)warp * hstride;
    const unsigned hsw_off = (unsigned)warp * (unsigned)hstride * 4u;        // byte offset of the warp's block

    FinishLane f;
    f.init(lane, warp, B);
    const bool fin_warp = warp < nu;

    // warps whose column range lies beyond H and that finish no unit leave now (their partial sums stay zero)
    const int n_active = (H + kspan - 1) / kspan;
    const int nbar = 32 * max(n_active, nu);
    if (warp * 32 >= nbar) return;

    int it = 0;
#pragma unroll 1
    for (int s = 0; s < T; ++s) {
        const int t = d ? (T - 1 - s) : s;
#pragma unroll 1
        for (int ci = 0; ci < nchunk; ++ci, ++it) {
            const int b0 = ci * kChunk;
            const int nb = min(kChunk, B - b0);
            // projection term of this lane's (batch row, gate): requested now, needed after the products
            float gv[kMaxSplit];
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp) gv[sp] = 0.0f;
            if (FUSE) {
                if (fin_warp && f.fpart == 0) gv[0] = G_s[(size_t)t * GP + warp * 4 + f.fq];
            } else if (fin_warp && f.fpart == 0 && b0 + f.fb < B) {
                const float *gp = a.G + (((size_t)t * B + b0 + f.fb) * D + d) * 4 * H + (size_t)(u0 + warp) * 4 + f.fq;
#pragma unroll
                for (int sp = 0; sp < kMaxSplit; ++sp)
                    if (sp < a.nsplit) gv[sp] = ld_nc_early(gp + (size_t)sp * a.g_split_stride);
            }

            // ---- this warp's columns of h_{t-1}, rows b0 .. b0+nb-1, into the staging rows
            const int nwords = nb * kspan;
            if (s == 0) {
                for (int idx = lane; idx < nwords; idx += 32) {
                    const int b = idx / kspan, kk = idx - b * kspan;
                    if (kbase + kk < H) hsw[idx] = a.h0 ? a.h0[((size_t)d * B + b0 + b) * H + kbase + kk] : 0.0f;
                }
            } else if (!(probe & kProbeNoExchange)) {
                const unsigned want = a.stamp_base + (unsigned)s;            // stamp of step s-1
                const unsigned long long *src = xch_d + ((size_t)((s - 1) & 1) * B + b0) * H;
                auto off = [&](int idx, long long &so, unsigned &wnt) -> bool {
                    int b = 0, kk = idx;
                    if (!ONE) { b = idx / kspan; kk = idx - b * kspan; }
                    so = b * H + kbase + kk;
                    wnt = want;
                    return kbase + kk < H;
                };
                auto sink = [&](int idx, float v) { hsw[idx] = v; };
                poll_words<4>(src, nwords, lane, off, sink, abort_v, a.spin_limit, a.status);
            }
            __syncwarp();

            // ---- the register list: one gather and two multiply-adds per entry and batch row
            // (accT: both rows together, accB: the second row; the first row is their difference)
            float accT[NB], accB[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) { accT[b] = 0.0f; accB[b] = 0.0f; }
            if (!(probe & kProbeNoProducts)) {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    unsigned w = ent[e];
                    asm volatile("" : "+r"(w));          // decode inside the step: decoded copies would triple the registers
                    const float v = __uint_as_float(w & 0xffff0000u);
                    const unsigned off = hsw_off | (w & 0x7ffcu);
                    const bool second = (w & 0x8000u) != 0;
                    if (!LSTM_CHECK_INDEX((w & 0x7ffcu) + (unsigned)((NB - 1) * kspan) * 4u, (unsigned)hstride * 4u, a.status)) continue;
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const float hv = *reinterpret_cast<const float *>(smem + off + (unsigned)(b * kspan) * 4u);
                        accT[b] = fmaf(v, hv, accT[b]);
                        if (second) accB[b] = fmaf(v, hv, accB[b]);
                    }
                }
            }
            float *rwp = red + (size_t)((it & 1) * NW + warp) * WS;
#pragma unroll
            for (int b = 0; b < NB; ++b)
                if (b < nb) {
                    if (rowA != 0xff) rwp[b * RP + rowA] = accT[b] - accB[b];
                    if (rowB != 0xff) rwp[b * RP + rowB] = accB[b];
                }

            // ---- all partial sums of this pass are in place (two barriers and two buffers alternate)
            bar_sync(1 + (it & 1), nbar);

            if (fin_warp && (probe & kProbeNoGates)) {
                if (f.fq == 0 && f.fpart == 0 && f.fb < nb && (int)blockIdx.x != a.withhold_cta)
                    st_relaxed_u64(xch_d + ((size_t)(s & 1) * B + b0 + f.fb) * H + u0 + warp,
                                   ((unsigned long long)(a.stamp_base + (unsigned)s + 1u) << 32) | 0x3e800000ull);
            } else if (fin_warp) {
                const int j = u0 + warp;
                const float z_in = (gv[0] + gv[1]) + (gv[2] + gv[3]);
                finish_unit<NW>(f, red + (size_t)((it & 1) * NW) * WS, RP, WS, nb, z_in, c_s + warp * B, b0, B, H, j,
                                a.stamp_base + (unsigned)s + 1u, xch_d + (size_t)(s & 1) * B * H,
                                (int)blockIdx.x != a.withhold_cta,
                                a.y + (size_t)t * B * D * H + (size_t)d * H + j, (size_t)D * H,
                                a.xb_next ? a.xb_next + (size_t)t * B * a.xb_ld + (size_t)d * H + j : nullptr, (size_t)a.xb_ld,
                                a.xb_plane, s == T - 1, a.hT ? a.hT + (size_t)d * B * H : nullptr,
                                a.cT ? a.cT + (size_t)d * B * H : nullptr);
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

typedef void (*KernelFn)(const RecurCsrArgs);

template <int NW, bool ONE, bool PROBE, bool FUSE = false>
KernelFn pick_slots(int slots)
{
    switch (slots) {
        case 8: return recur_csr_kernel<8, NW, ONE, PROBE, FUSE>;
        case 16: return recur_csr_kernel<16, NW, ONE, PROBE, FUSE>;
        case 20: return recur_csr_kernel<20, NW, ONE, PROBE, FUSE>;
        case 24: return recur_csr_kernel<24, NW, ONE, PROBE, FUSE>;
        case 28: return recur_csr_kernel<28, NW, ONE, PROBE, FUSE>;
        case 32: return recur_csr_kernel<32, NW, ONE, PROBE, FUSE>;
        case 40: return recur_csr_kernel<40, NW, ONE, PROBE, FUSE>;
        case 48: return recur_csr_kernel<48, NW, ONE, PROBE, FUSE>;
        case 64: return recur_csr_kernel<64, NW, ONE, PROBE, FUSE>;
        default: return nullptr;
    }
}
template <bool ONE, bool PROBE>
KernelFn pick_nw(int slots, int nw)
{
    if (nw == 16) return pick_slots<16, ONE, PROBE>(slots);
    if (nw == 8) {
        if (slots == 96) return recur_csr_kernel<96, 8, ONE, PROBE>;
        if (slots == 128) return recur_csr_kernel<128, 8, ONE, PROBE>;
        return pick_slots<8, ONE, PROBE>(slots);
    }
    return nullptr;
}
// variant 0: up to four sequences per pass, 1: one sequence, 2: the measurement build of 1, 3: one sequence with
// the projection in the prologue (16 warps only)
KernelFn pick(int slots, int nw, int variant)
{
    if (variant == 0) return pick_nw<false, false>(slots, nw);
    if (variant == 1) return pick_nw<true, false>(slots, nw);
    if (variant == 3) return nw == 16 ? pick_slots<16, true, false, true>(slots) : nullptr;
    return pick_nw<true, true>(slots, nw);
}

}  // namespace

int recur_csr_reg_slots(int needed, int nw)
{
    static const int built[] = {8, 16, 20, 24, 28, 32, 40, 48, 64, 96, 128};
    const int cap = nw == 16 ? kCsrRegMaxSlots16 : nw == 8 ? kCsrRegMaxSlots8 : 0;
    for (int v : built)
        if (v >= needed && v <= cap) return v;
    return 0;
}

int recur_csr_reg_hs_stride(int kspan, int B)
{
    const int need = (B == 1 ? 1 : kChunk) * kspan;
    int s = 32;
    while (s < need) s <<= 1;
    return s;
}

size_t recur_csr_reg_smem_bytes(int nw, int kspan, int mt, int upc, int B)
{
    return ((size_t)nw * recur_csr_reg_hs_stride(kspan, B) + (size_t)2 * nw * red_warp_pitch(mt) + (size_t)((upc * B + 3) & ~3)) * 4;
}

// fused projection: the partial products of all warps (24 timesteps x rows each) lie over the kernel's other
// shared memory, the finished rows of G behind whichever is larger
size_t recur_csr_reg_fuse_gs_offset(int nw, int kspan, int mt, int upc)
{
    const size_t normal = recur_csr_reg_smem_bytes(nw, kspan, mt, upc, 1);
    const size_t partial = (size_t)nw * 24 * (mt * 16 + 1) * 4;
    return (std::max(normal, partial) + 15) & ~(size_t)15;
}
size_t recur_csr_reg_fuse_smem_bytes(int nw, int kspan, int mt, int upc)
{
    return recur_csr_reg_fuse_gs_offset(nw, kspan, mt, upc) + (size_t)kFuseMaxT * (mt * 16 + 1) * 4;
}

cudaError_t recur_csr_reg_prepare(int slots, int nw, int max_smem)
{
    for (int variant = 0; variant < 4; ++variant) {
        KernelFn fn = pick(slots, nw, variant);
        if (!fn && variant == 3) continue;                      // no fused build for this warp count
        if (!fn) return cudaErrorInvalidValue;
        const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_recur_csr_reg(const RecurCsrArgs &a, int slots, int nw, size_t smem, cudaStream_t st)
{
    int variant = a.B == 1 ? 1 : 0;
    if (a.fuse) {
        if (a.B != 1 || a.probe || nw != 16 || a.T > kFuseMaxT) return cudaErrorInvalidValue;
        variant = 3;
    }
    if (a.probe) {
        if (variant != 1) return cudaErrorInvalidValue;
        variant = 2;
    }
    KernelFn fn = pick(slots, nw, variant);
    if (!fn) return cudaErrorInvalidValue;
    RecurCsrArgs copy = a;
    copy.hs_stride = recur_csr_reg_hs_stride(a.kspan, a.B);
    void *params[] = {&copy};
    return cudaLaunchCooperativeKernel((const void *)fn, dim3(a.ncta_dir * (a.ndirs ? a.ndirs : a.D)), dim3(nw * 32), params, smem, st);
}

}  // namespace lstm
