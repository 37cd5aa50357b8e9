// Layer-wavefront recurrent kernel for unidirectional stacks with bf16 weights: ALL layers of the stack in
// one persistent launch, layer l working on timestep t while layer l-1 already works on t+1 (paper, Section
// 5.1: the language model is two stacked recurrent layers; Section 4 gives the cell).  A stack of L layers and
// T steps then costs T + L - 1 serial steps instead of L * T, and the input projections of the layers above the
// first -- which cannot be hoisted out of the time loop once the layers overlap -- are folded into the step:
// layer l >= 1 multiplies the concatenation [h^{l-1}_t ; h^l_{t-1}] by its [Wx_l | Wh_l], exactly the
// W [x_t, h_{t-1}] of the paper's cell equations.  Layer 0 still takes its input half from the projection
// computed for all timesteps beforehand.
//
// Design.  The SMs are split evenly between the layers; inside a layer's group the structure is the dense
// register-resident kernel's: a CTA owns a contiguous range of hidden units with all four gate rows, its slice
// of the layer's matrix lives in registers (and, beyond the register budget, in shared memory) as operand-A
// fragments of mma.sync.m16n8k16, warp w owns a column range of the concatenated operand, and after one CTA
// barrier warp w finishes unit w.  Every layer publishes h_t as stamped 64-bit words into its own buffer with
// one slot per TIMESTEP (not two alternating ones): the layer below may run any number of steps ahead of the
// layer above, so a slot must not be reused within a call.  A warp polls the words of its column range from
// two places: columns below H from the lower layer's slot t, the others from its own layer's slot t-1; both
// in one polling round, each word with the stamp it must carry.
// Every wait is bounded: when it expires the CTA records a timeout status, stops waiting and runs to the end.
#include "common.cuh"
#include "device_util.cuh"
#include "recur_parts.cuh"

namespace lstm {
namespace {

constexpr int kMaxSplit = 4;

// MT: 16-row tiles per CTA; NKR: 16-column tiles per warp held in registers; NW: warps per CTA;
// ONE: a single sequence (B = 1).
template <int MT, int NKR, int NW, bool ONE>
__global__ void __launch_bounds__(NW * 32, 1) recur_wave_kernel(const RecurWaveArgs a)
{
    constexpr int NT = NW * 32;
    constexpr int RP = red_row_pitch(MT), WS = red_warp_pitch(MT);
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int abort_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int H = a.H, B = ONE ? 1 : a.B, T = a.T;
    const int layer = blockIdx.x / a.ncta_layer;
    const int cta = blockIdx.x % a.ncta_layer;
    int u0, nu;
    unit_range(H, a.ncta_layer, cta, u0, nu);
    const int upc = (H + a.ncta_layer - 1) / a.ncta_layer;
    const int K = layer == 0 ? H : 2 * H;              // columns of this layer's operand: [h below ; own h]
    const int lowk = layer == 0 ? 0 : H;               // columns [0, lowk) come from the layer below
    const int nkw = a.nkw[layer];                      // column tiles per warp, >= NKR
    const int nks = nkw - NKR;
    const int kspan = nkw * 16, kbase = warp * kspan;
    const int nkw_max = a.nkw_max;

    // ---- shared-memory carve-up (sized for the layer with the most column tiles)
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem);                  // [NW][nkw][8][16]
    float *red = reinterpret_cast<float *>(smem + (size_t)NW * nkw_max * 256);    // [2][NW][WS]
    float *c_s = red + 2 * NW * WS;                                               // [upc][B]
    uint4 *As = reinterpret_cast<uint4 *>(c_s + ((upc * B + 3) & ~3));            // [NW][nks][MT][32]
    LSTM_CHECK_SMEM_END((size_t)(reinterpret_cast<unsigned char *>(As + (size_t)NW * (nkw_max - NKR) * MT * 32) - smem), a.status);

    // ---- residency: this warp's tiles, registers first, the rest in shared memory
    const uint4 *wsrc = a.wfrag[layer] + ((size_t)(cta * NW + warp) * nkw) * MT * 32 + lane;
    uint4 areg[NKR][MT];
#pragma unroll
    for (int i = 0; i < NKR; ++i)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) areg[i][mt] = __ldg(wsrc + (size_t)(i * MT + mt) * 32);
    uint4 *As_w = As + (size_t)warp * nks * MT * 32 + lane;
    for (int i = 0; i < nks * MT; ++i) As_w[(size_t)i * 32] = __ldg(wsrc + (size_t)(NKR * MT + i) * 32);

    for (int i = tid; i < NW * nkw_max * 64; i += NT) reinterpret_cast<unsigned *>(Bs)[i] = 0u;
    for (int i = tid; i < 2 * NW * WS; i += NT) red[i] = 0.0f;
    const float *c0 = a.c0 ? a.c0 + (size_t)layer * B * H : nullptr;
    const float *h0 = a.h0 ? a.h0 + (size_t)layer * B * H : nullptr;
    for (int i = tid; i < nu * B; i += NT) {
        const int u = i / B, b = i - u * B;
        c_s[u * B + b] = c0 ? c0[(size_t)b * H + u0 + u] : 0.0f;
    }
    if (tid == 0) abort_s = 0;
    __syncthreads();
    volatile int *abort_v = &abort_s;

    // exchange buffers: one slot of [B][H] words per (layer, timestep)
    unsigned long long *xch_own = a.xch + (size_t)layer * T * B * H;
    const unsigned long long *xch_low = layer > 0 ? a.xch + (size_t)(layer - 1) * T * B * H : nullptr;
    __nv_bfloat16 *Bw = Bs + (size_t)warp * nkw * 128;
    const unsigned *Bw32 = reinterpret_cast<const unsigned *>(Bw);

    FinishLane f;
    f.init(lane, warp, B);
    const bool fin_warp = warp < nu;
    // layers above the first: the bias of this lane's (unit, gate) stands where layer 0 has the projection term
    float bias_v = 0.0f;
    if (layer > 0 && fin_warp && a.bias[layer]) bias_v = __ldg(a.bias[layer] + (size_t)(u0 + warp) * 4 + f.fq);

    const int n_active = (K + kspan - 1) / kspan;
    const int nbar = 32 * max(n_active, nu);
    if (warp * 32 >= nbar) return;

    const int nwords = B * kspan;
#pragma unroll 1
    for (int s = 0; s < T; ++s) {
        // input term of this lane's (batch row, gate): requested now, needed after the products
        float gv[kMaxSplit];
#pragma unroll
        for (int sp = 0; sp < kMaxSplit; ++sp) gv[sp] = 0.0f;
        if (layer == 0 && fin_warp && f.fpart == 0 && f.fb < B) {
            const float *gp = a.G + ((size_t)s * B + f.fb) * 4 * H + (size_t)(u0 + warp) * 4 + f.fq;
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp)
                if (sp < a.nsplit) gv[sp] = ld_nc_early(gp + (size_t)sp * a.g_split_stride);
        }

        // ---- this warp's columns of [h^{l-1}_s ; h^l_{s-1}] as bf16 hi/lo parts in operand-B order
        auto put = [&](int idx, float v) {
            int b = 0, kk = idx;
            if (!ONE) { b = idx / kspan; kk = idx - b * kspan; }
            const int dof = ((kk >> 4) * 8 + 2 * b) * 16 + (kk & 15);
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            if (!LSTM_CHECK_INDEX(dof + 16, nkw * 128, a.status)) return;
            Bw[dof] = hi;
            Bw[dof + 16] = __float2bfloat16_rn(v - __bfloat162float(hi));
        };
        if (s == 0) {
            // the own-layer half is the initial state
            for (int idx = lane; idx < nwords; idx += 32) {
                int b = 0, kk = idx;
                if (!ONE) { b = idx / kspan; kk = idx - b * kspan; }
                const int k = kbase + kk;
                if (k >= lowk && k < K) put(idx, h0 ? h0[(size_t)b * H + (k - lowk)] : 0.0f);
            }
        }
        {
            const unsigned want_low = a.stamp_base + (unsigned)s + 1u;      // the layer below has published step s
            const unsigned want_own = a.stamp_base + (unsigned)s;           // this layer has published step s-1
            auto off = [&](int idx, long long &so, unsigned &wnt) -> bool {
                int b = 0, kk = idx;
                if (!ONE) { b = idx / kspan; kk = idx - b * kspan; }
                const int k = kbase + kk;
                if (k >= K) return false;
                if (k < lowk) {
                    so = (xch_low - a.xch) + ((long long)s * B + b) * H + k;
                    wnt = want_low;
                    return true;
                }
                if (s == 0) return false;
                so = (xch_own - a.xch) + ((long long)(s - 1) * B + b) * H + (k - lowk);
                wnt = want_own;
                return true;
            };
            poll_words<4>(a.xch, nwords, lane, off, put, abort_v, a.spin_limit, a.status);
        }
        __syncwarp();

        // ---- partial products of this warp's columns: registers first, then the shared-memory tiles
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
        for (int i = 0; i < nks; ++i) {
            const unsigned bv0 = Bw32[(NKR + i) * 64 + g * 8 + tig];
            const unsigned bv1 = Bw32[(NKR + i) * 64 + g * 8 + tig + 4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) mma_bf16(acc[mt], As_w[(size_t)(i * MT + mt) * 32], bv0, bv1);
        }
        // accumulator columns 2*tig and 2*tig+1 are the hi and lo parts of batch row tig
        float *rw = red + (size_t)((s & 1) * NW + warp) * WS + tig * RP + g;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            rw[mt * 16] = acc[mt][0] + acc[mt][1];
            rw[mt * 16 + 8] = acc[mt][2] + acc[mt][3];
        }

        bar_sync(1 + (s & 1), nbar);

        if (fin_warp) {
            const int j = u0 + warp;
            const float z_in = layer == 0 ? (gv[0] + gv[1]) + (gv[2] + gv[3]) : bias_v;
            const bool top = layer == a.L - 1;
            finish_unit<NW>(f, red + (size_t)((s & 1) * NW) * WS, RP, WS, B, z_in, c_s + warp * B, 0, B, H, j,
                            a.stamp_base + (unsigned)s + 1u, xch_own + (size_t)s * B * H, (int)blockIdx.x != a.withhold_cta,
                            top ? a.y + (size_t)s * B * H + j : nullptr, (size_t)H, nullptr, 0, 0, s == T - 1,
                            a.hT ? a.hT + (size_t)layer * B * H : nullptr, a.cT ? a.cT + (size_t)layer * B * H : nullptr);
        }
        // Warps that finish no unit must not start to poll before this CTA has issued its own stores.
        if (nbar > 32 * nu) {
            if (fin_warp) bar_arrive(3 + (s & 1), nbar);
            else bar_sync(3 + (s & 1), nbar);
        }
    }
}

typedef void (*KernelFn)(const RecurWaveArgs);

template <int MT, bool ONE>
KernelFn pick_nkr(int nkr)
{
    switch (nkr) {
        case 2: return recur_wave_kernel<MT, 2, 16, ONE>;
        case 4: return recur_wave_kernel<MT, 4, 16, ONE>;
        case 6: return recur_wave_kernel<MT, 6, 16, ONE>;
        case 8: return recur_wave_kernel<MT, 8, 16, ONE>;
        default: return nullptr;
    }
}
template <bool ONE>
KernelFn pick_mt(int mt, int nkr)
{
    switch (mt) {
        case 1: return pick_nkr<1, ONE>(nkr);
        case 2: return pick_nkr<2, ONE>(nkr);
        case 3: return pick_nkr<3, ONE>(nkr);
        case 4: return pick_nkr<4, ONE>(nkr);
        default: return nullptr;
    }
}
KernelFn pick(int mt, int nkr, bool one)
{
    if (mt < 1 || mt > 4 || mt * nkr > kWaveTileCap) return nullptr;
    return one ? pick_mt<true>(mt, nkr) : pick_mt<false>(mt, nkr);
}

}  // namespace

bool recur_wave_shape_ok(int mt, int nkr) { return pick(mt, nkr, true) != nullptr; }

size_t recur_wave_smem_bytes(int mt, int nkr, int nkw_max, int upc, int B)
{
    const int nw = 16;
    return (size_t)nw * nkw_max * 256 + (size_t)2 * nw * red_warp_pitch(mt) * 4 + (size_t)((upc * B + 3) & ~3) * 4 +
           (size_t)nw * (nkw_max - nkr) * mt * 512;
}

cudaError_t recur_wave_prepare(int mt, int nkr, int max_smem)
{
    for (int one = 0; one < 2; ++one) {
        KernelFn fn = pick(mt, nkr, one != 0);
        if (!fn) return cudaErrorInvalidValue;
        const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_recur_wave(const RecurWaveArgs &a, int mt, int nkr, size_t smem, cudaStream_t st)
{
    KernelFn fn = pick(mt, nkr, a.B == 1);
    if (!fn) return cudaErrorInvalidValue;
    RecurWaveArgs copy = a;
    void *params[] = {&copy};
    return cudaLaunchCooperativeKernel((const void *)fn, dim3(a.ncta_layer * a.L), dim3(16 * 32), params, smem, st);
}

}  // namespace lstm
