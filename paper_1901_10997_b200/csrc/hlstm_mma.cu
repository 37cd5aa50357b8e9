// Recurrent kernel of the H-LSTM cell for bf16 weights: the paper's Section 4 cell equations with ONE
// hidden layer (linear map + ReLU) inside each gate.  Per step, for gate q in {i,f,g,o}:
//     r_q = relu(P[t]_q + Uh_q h_{t-1})          P[t] = a + Ux x_t, the input half, computed beforehand
//     z_q = b_q + W_q r_q
//     i,f,o = sigmoid(z_i,z_f,z_o), g = tanh(z_g);  c_t = f c_{t-1} + i g;  h_t = o tanh(c_t)
//
// Same structure as the register-resident LSTM kernel (recur_mma.cu): one cooperative launch per layer,
// CTAs own contiguous ranges of units, weights stay on-chip as operand-A fragments of mma.m16n8k16,
// values travel between CTAs as stamped 64-bit words that the consumers poll, every wait is bounded.
// A step has two passes, each with its own exchange:
//   pass 1: the CTA's rows of the four Uh_q (its hidden units, fragments in REGISTERS) times h_{t-1}
//           (bf16 hi + lo in operand-B columns 0, 1); relu; the 4 values of a hidden unit are published;
//   pass 2: the CTA's rows of the four W_q (its cell units, fragments in SHARED memory) times r_i..r_o,
//           which sit side by side in the operand-B columns (gate q -> columns 2q, 2q+1), so the one
//           instruction stream serves four different right-hand sides; gate functions, c/h update, h is
//           published.
// Batch rows are processed one after the other (two passes each).
#include "common.cuh"
#include "device_util.cuh"

namespace lstm {
namespace {





constexpr int kPoll = 4;
constexpr int kMaxSplit = 4;

// Polls this warp's columns [kbase, kbase + kspan) of `rows` vectors of length K (row r starts at
// src + r * row_stride) until every word carries the stamp `want`, and stages the values as bf16 hi/lo
// parts: row r -> operand-B columns 2r, 2r+1.  Returns when done or when the CTA has given up.
__device__ __forceinline__ void poll_and_stage(const unsigned long long *src, int rows, int row_stride, int K,
                                               int kbase, int kspan, unsigned want, __nv_bfloat16 *Bw, int lane,
                                               volatile int *abort_v, int *status, long long spin_limit)
{
    const int nwords = rows * kspan;
    long long t_start = 0;
    for (int base = 0; base < nwords; base += 32 * kPoll) {
        unsigned pending = 0;
        int soff[kPoll], doff[kPoll];
#pragma unroll
        for (int i = 0; i < kPoll; ++i) {
            const int idx = base + lane + 32 * i;
            const int r = (idx >= kspan) + (idx >= 2 * kspan) + (idx >= 3 * kspan), kk = idx - r * kspan;
            soff[i] = r * row_stride + kbase + kk;
            doff[i] = ((kk >> 4) * 8 + 2 * r) * 16 + (kk & 15);
            if (idx < nwords && kbase + kk < K) pending |= 1u << i;
        }
        if (*abort_v) pending = 0;
        int rounds = 0;
        while (pending) {
            unsigned long long w[kPoll];
#pragma unroll
            for (int i = 0; i < kPoll; ++i)
                if (pending & (1u << i)) w[i] = ld_relaxed_u64(src + soff[i]);
#pragma unroll
            for (int i = 0; i < kPoll; ++i)
                if ((pending & (1u << i)) && (unsigned)(w[i] >> 32) == want) {
                    const float v = __uint_as_float((unsigned)w[i]);
                    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                    Bw[doff[i]] = hi;
                    Bw[doff[i] + 16] = __float2bfloat16_rn(v - __bfloat162float(hi));
                    pending &= ~(1u << i);
                }
            if (pending && ((++rounds & 63) == 0)) {
                const long long now = clock64();
                if (t_start == 0) t_start = now;
                if (*abort_v) pending = 0;
                else if (now - t_start > spin_limit || ld_volatile_s32(status) != kStatusOk) {
                    *abort_v = 1;
                    atomicExch(status, kStatusTimeout);
                    pending = 0;
                }
            }
        }
    }
}

// MT: 16-row tiles per CTA (covers 4 x hidden units and 4 x cell units of a CTA); NKR: pass-1 column
// tiles per warp in registers; NW: warps per CTA.
template <int MT, int NKR, int NW>
__global__ void __launch_bounds__(NW * 32, 1) hlstm_mma_kernel(const HlstmArgs a)
{
    constexpr int NT = NW * 32;
    constexpr int RP = MT * 16 + 8;
    constexpr int WS = 4 * RP + 4;
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int abort_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int H = a.H, Hh = a.Hh, B = a.B, T = a.T, D = a.D;
    const int d = a.dir0 + blockIdx.x / a.ncta_dir;
    const int cta = blockIdx.x % a.ncta_dir;
    int m0, nm, u0, nu;
    unit_range(Hh, a.ncta_dir, cta, m0, nm);       // hidden units of this CTA (pass 1)
    unit_range(H, a.ncta_dir, cta, u0, nu);        // cell units of this CTA (pass 2)
    const int upc = (H + a.ncta_dir - 1) / a.ncta_dir;
    const int nks1 = a.nks1, nkw1 = NKR + nks1, nkw2 = a.nkw2;
    const int kspan1 = nkw1 * 16, kbase1 = warp * kspan1;
    const int kspan2 = nkw2 * 16, kbase2 = warp * kspan2;
    const int nkwb = max(nkw1, nkw2);

    // ---- shared-memory carve-up
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem);                   // [NW][nkwb][8][16]
    float *red = reinterpret_cast<float *>(smem + (size_t)NW * nkwb * 256);        // [2][NW][WS]
    float *c_s = red + 2 * NW * WS;                                                // [upc][B]
    uint4 *As1 = reinterpret_cast<uint4 *>(c_s + ((upc * B + 3) & ~3));            // [NW][nks1][MT][32]
    uint4 *As2 = As1 + (size_t)NW * nks1 * MT * 32;                                // [NW][nkw2][MT][32]

    // ---- residency
    const uint4 *w1 = a.frag1[d] + ((size_t)(cta * NW + warp) * nkw1) * MT * 32 + lane;
    uint4 areg[NKR][MT];
#pragma unroll
    for (int i = 0; i < NKR; ++i)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) areg[i][mt] = __ldg(w1 + (size_t)(i * MT + mt) * 32);
    uint4 *As1_w = As1 + (size_t)warp * nks1 * MT * 32 + lane;
    for (int i = 0; i < nks1 * MT; ++i) As1_w[(size_t)i * 32] = __ldg(w1 + (size_t)(NKR * MT + i) * 32);
    const uint4 *w2 = a.frag2[d] + ((size_t)(cta * NW + warp) * nkw2) * MT * 32 + lane;
    uint4 *As2_w = As2 + (size_t)warp * nkw2 * MT * 32 + lane;
    for (int i = 0; i < nkw2 * MT; ++i) As2_w[(size_t)i * 32] = __ldg(w2 + (size_t)i * 32);

    for (int i = tid; i < NW * nkwb * 64; i += NT) reinterpret_cast<unsigned *>(Bs)[i] = 0u;
    for (int i = tid; i < 2 * NW * WS; i += NT) red[i] = 0.0f;
    for (int i = tid; i < nu * B; i += NT) {
        const int u = i / B, b = i - u * B;
        c_s[u * B + b] = a.c0 ? a.c0[((size_t)d * B + b) * H + u0 + u] : 0.0f;
    }
    if (tid == 0) abort_s = 0;
    __syncthreads();
    volatile int *abort_v = &abort_s;

    unsigned long long *xch_d = a.xch + (size_t)d * 2 * B * H;            // h words   [2][B][H]
    unsigned long long *rxch_d = a.rxch + (size_t)d * 2 * B * 4 * Hh;     // r words   [2][B][4][Hh]
    __nv_bfloat16 *Bw = Bs + (size_t)warp * nkwb * 128;
    const unsigned *Bw32 = reinterpret_cast<const unsigned *>(Bw);

    // finishing role: warp w finishes hidden unit w in pass 1 and cell unit w in pass 2; the 32 lanes are
    // 4 gates x 8 lanes that share the sum over the warps' partial results
    const int fq = lane >> 3, fpart = lane & 7;
    const int frow = warp * 4 + fq;
    const bool fin1 = warp < nm, fin2 = warp < nu;
    const float b_out = (fin2 && fpart == 0 && a.bias_out) ? a.bias_out[((size_t)d * H + u0 + warp) * 4 + fq] : 0.0f;

    const int n_act = max((H + kspan1 - 1) / kspan1, (Hh + kspan2 - 1) / kspan2);
    const int nbar = 32 * max(n_act, max(nm, nu));
    if (warp * 32 >= nbar) return;

    int it = 0;
#pragma unroll 1
    for (int s = 0; s < T; ++s) {
        const int t = d ? (T - 1 - s) : s;
        const unsigned stamp = a.stamp_base + (unsigned)s + 1u;           // of everything published in step s
#pragma unroll 1
        for (int b = 0; b < B; ++b) {
            // ======================= pass 1: hidden layers of the four gates =======================
            float gp[kMaxSplit];
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp) gp[sp] = 0.0f;
            if (fin1 && fpart == 0) {
                const float *p = a.G + (((size_t)t * B + b) * D + d) * 4 * Hh + (size_t)(m0 + warp) * 4 + fq;
#pragma unroll
                for (int sp = 0; sp < kMaxSplit; ++sp)
                    if (sp < a.nsplit) gp[sp] = ld_nc_early(p + (size_t)sp * a.g_split_stride);
            }
            if (s == 0) {
                for (int kk = lane; kk < kspan1; kk += 32) {
                    const int k = kbase1 + kk;
                    if (k < H) {
                        const float v = a.h0 ? a.h0[((size_t)d * B + b) * H + k] : 0.0f;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                        const int o = (kk >> 4) * 128 + (kk & 15);
                        Bw[o] = hi;
                        Bw[o + 16] = __float2bfloat16_rn(v - __bfloat162float(hi));
                    }
                }
            } else {
                poll_and_stage(xch_d + ((size_t)((s - 1) & 1) * B + b) * H, 1, 0, H, kbase1, kspan1, stamp - 1u, Bw, lane,
                               abort_v, a.status, a.spin_limit);
            }
            __syncwarp();
            {
                float acc[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
#pragma unroll
                for (int i = 0; i < NKR; ++i) {
                    const unsigned bv0 = Bw32[i * 64 + g * 8 + tig];
                    const unsigned bv1 = Bw32[i * 64 + g * 8 + tig + 4];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], areg[i][mt], bv0, bv1);
                }
                for (int i = 0; i < nks1; ++i) {
                    const unsigned bv0 = Bw32[(NKR + i) * 64 + g * 8 + tig];
                    const unsigned bv1 = Bw32[(NKR + i) * 64 + g * 8 + tig + 4];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], As1_w[(size_t)(i * MT + mt) * 32], bv0, bv1);
                }
                float *rw = red + (size_t)((it & 1) * NW + warp) * WS + tig * RP + g;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    rw[mt * 16] = acc[mt][0] + acc[mt][1];
                    rw[mt * 16 + 8] = acc[mt][2] + acc[mt][3];
                }
            }
            bar_sync(1 + (it & 1), nbar);
            if (fin1) {
                // columns 0, 1 of the operand hold h: partial sums of "row" 0
                float z = 0.0f;
                const float *rp = red + (size_t)((it & 1) * NW) * WS + frow;
                for (int w = fpart; w < NW; w += 8) z += rp[(size_t)w * WS];
                z += __shfl_xor_sync(0xffffffffu, z, 4);
                z += __shfl_xor_sync(0xffffffffu, z, 2);
                z += __shfl_xor_sync(0xffffffffu, z, 1);
                z += (gp[0] + gp[1]) + (gp[2] + gp[3]);
                const float r = fmaxf(z, 0.0f);
                if (fpart == 0 && (int)blockIdx.x != a.withhold_cta)
                    st_relaxed_u64(rxch_d + (((size_t)(s & 1) * B + b) * 4 + fq) * Hh + m0 + warp,
                                   ((unsigned long long)stamp << 32) | (unsigned long long)__float_as_uint(r));
            }
            if (nbar > 32 * nm) {
                if (fin1) bar_arrive(3 + (it & 1), nbar);
                else bar_sync(3 + (it & 1), nbar);
            }
            ++it;

            // ======================= pass 2: gate pre-activations from the hidden layers =======================
            poll_and_stage(rxch_d + ((size_t)(s & 1) * B + b) * 4 * Hh, 4, Hh, Hh, kbase2, kspan2, stamp, Bw, lane,
                           abort_v, a.status, a.spin_limit);
            __syncwarp();
            {
                float acc[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[mt][e] = 0.0f;
                for (int i = 0; i < nkw2; ++i) {
                    const unsigned bv0 = Bw32[i * 64 + g * 8 + tig];
                    const unsigned bv1 = Bw32[i * 64 + g * 8 + tig + 4];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], As2_w[(size_t)(i * MT + mt) * 32], bv0, bv1);
                }
                // accumulator columns 2*tig, 2*tig+1: hi and lo parts of r of gate tig
                float *rw = red + (size_t)((it & 1) * NW + warp) * WS + tig * RP + g;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    rw[mt * 16] = acc[mt][0] + acc[mt][1];
                    rw[mt * 16 + 8] = acc[mt][2] + acc[mt][3];
                }
            }
            bar_sync(1 + (it & 1), nbar);
            if (fin2) {
                // row 4u+q of W belongs to gate q: its sum against r_q sits in "row" q of the partial sums
                float z = 0.0f;
                const float *rp = red + (size_t)((it & 1) * NW) * WS + fq * RP + frow;
                for (int w = fpart; w < NW; w += 8) z += rp[(size_t)w * WS];
                z += __shfl_xor_sync(0xffffffffu, z, 4);
                z += __shfl_xor_sync(0xffffffffu, z, 2);
                z += __shfl_xor_sync(0xffffffffu, z, 1);
                z += b_out;
                // one expression for both gate functions: logistic, or tanh z = 2 logistic(2z) - 1 for the candidate
                const float act = fmaf(fq == 2 ? 2.0f : 1.0f,
                                       __fdividef(1.0f, 1.0f + ex2_fast((fq == 2 ? -2.8853900817779268f : -1.4426950408889634f) * z)),
                                       fq == 2 ? -1.0f : 0.0f);
                const float vi = __shfl_sync(0xffffffffu, act, 0);
                const float vf = __shfl_sync(0xffffffffu, act, 8);
                const float vg = __shfl_sync(0xffffffffu, act, 16);
                const float vo = __shfl_sync(0xffffffffu, act, 24);
                if (lane == 0) {
                    const int j = u0 + warp;
                    const float cn = fmaf(vf, c_s[warp * B + b], vi * vg);
                    const float hn = vo * tanh_fast(cn);
                    if ((int)blockIdx.x != a.withhold_cta)
                        st_relaxed_u64(xch_d + ((size_t)(s & 1) * B + b) * H + j,
                                       ((unsigned long long)stamp << 32) | (unsigned long long)__float_as_uint(hn));
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
            if (nbar > 32 * nu) {
                if (fin2) bar_arrive(3 + (it & 1), nbar);
                else bar_sync(3 + (it & 1), nbar);
            }
            ++it;
        }
    }
}

typedef void (*KernelFn)(const HlstmArgs);

template <int MT, int NW>
KernelFn pick_nkr(int nkr)
{
    switch (nkr) {
        case 2: return hlstm_mma_kernel<MT, 2, NW>;
        case 4: return hlstm_mma_kernel<MT, 4, NW>;
        case 6: return hlstm_mma_kernel<MT, 6, NW>;
        case 8: return hlstm_mma_kernel<MT, 8, NW>;
        default: return nullptr;
    }
}
template <int NW>
KernelFn pick_mt(int mt, int nkr)
{
    switch (mt) {
        case 1: return pick_nkr<1, NW>(nkr);
        case 2: return pick_nkr<2, NW>(nkr);
        case 3: return pick_nkr<3, NW>(nkr);
        case 4: return pick_nkr<4, NW>(nkr);
        default: return nullptr;
    }
}
KernelFn pick(int mt, int nkr, int nw)
{
    if (!recur_mma_shape_ok(mt, nkr, nw)) return nullptr;
    return nw == 8 ? pick_mt<8>(mt, nkr) : pick_mt<16>(mt, nkr);
}

}  // namespace

size_t hlstm_mma_smem_bytes(int mt, int nkr, int nw, int nks1, int nkw2, int upc, int B)
{
    const int nkwb = (nkr + nks1) > nkw2 ? (nkr + nks1) : nkw2;
    return (size_t)nw * nkwb * 256 + (size_t)2 * nw * (4 * (mt * 16 + 8) + 4) * 4 + (size_t)((upc * B + 3) & ~3) * 4 +
           (size_t)nw * (nks1 + nkw2) * mt * 512;
}

cudaError_t hlstm_mma_prepare(int mt, int nkr, int nw, int max_smem)
{
    KernelFn fn = pick(mt, nkr, nw);
    if (!fn) return cudaErrorInvalidValue;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

cudaError_t launch_hlstm_mma(const HlstmArgs &a, int mt, int nkr, int nw, size_t smem, cudaStream_t st)
{
    KernelFn fn = pick(mt, nkr, nw);
    if (!fn) return cudaErrorInvalidValue;
    HlstmArgs copy = a;
    void *params[] = {&copy};
    return cudaLaunchCooperativeKernel((const void *)fn, dim3(a.ncta_dir * (a.ndirs ? a.ndirs : a.D)), dim3(nw * 32), params, smem, st);
}

}  // namespace lstm
