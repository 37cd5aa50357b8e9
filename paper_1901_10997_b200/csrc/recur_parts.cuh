// Parts of a recurrent step shared by the register-resident kernels that were written after the dense one
// (the sparse kernel and the layer-wavefront kernel): the bounded poll of stamped exchange words and the
// finishing role that turns per-warp partial sums into gates, state and the published h.
//
// Exchange protocol (same as the dense kernel's): h_t[b][j] of a direction travels as one 64-bit word
// {step stamp : 32 | value bits : 32} in xch[parity][b][j]; a consumer polls the word itself, so a step
// costs one L2 round trip after the last producer's store and needs no grid barrier.  Every poll is bounded
// by clock ticks; on expiry the CTA records a timeout in the status word, raises its abort flag and stops
// waiting for the rest of the launch.
#pragma once
#include "common.cuh"
#include "device_util.cuh"

namespace lstm {

// Polls the words idx = lane, lane + 32, ... < nwords of one pass, KP per lane in flight per round trip.
// off(idx, &word_offset, &stamp) says where word idx lives relative to src, which stamp it must carry, and
// whether it exists at all; sink(idx, value) receives every value once, as soon as its stamp is the wanted one.
template <int KP, class OffFn, class Sink>
__device__ __forceinline__ void poll_words(const unsigned long long *src, int nwords, int lane, OffFn off,
                                           Sink sink, volatile int *abort_v, long long spin_limit, int *status)
{
    long long t_start = 0;
    for (int base = 0; base < nwords; base += 32 * KP) {
        unsigned pending = 0;
        long long soff[KP];
        unsigned want[KP];
#pragma unroll
        for (int i = 0; i < KP; ++i) {
            const int idx = base + lane + 32 * i;
            soff[i] = 0; want[i] = 0;
            if (idx < nwords && off(idx, soff[i], want[i])) pending |= 1u << i;
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
                if ((pending & (1u << i)) && (unsigned)(w[i] >> 32) == want[i]) {
                    sink(base + lane + 32 * i, __uint_as_float((unsigned)w[i]));
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

// Layout of the per-warp partial sums of one pass: red[buffer][warp][batch row of the pass][local row], with
// pitches that keep the writers and the readers of a row on different banks.
__host__ __device__ constexpr int red_row_pitch(int mt) { return mt * 16 + 8; }
__host__ __device__ constexpr int red_warp_pitch(int mt) { return 4 * red_row_pitch(mt) + 4; }

// Finishing role of warp `warp` for unit `warp` of its CTA.  The 32 lanes form nbe * 4 (batch row, gate)
// groups of P = 8 / nbe lanes (nbe = 1, 2 or 4 batch rows a pass is laid out for); a group adds the NW warps'
// partial sums of its row, lane 0 of the group adds the input term and applies the gate function, and the
// lane of gate i updates c and h, publishes h as a stamped word and writes the outputs.
struct FinishLane {
    int P, fpart, fb, fq, frow;
    float act_k, act_sc, act_of;
    __device__ __forceinline__ void init(int lane, int warp, int B)
    {
        const int nbe = B >= 3 ? 4 : B;
        P = 8 / nbe;
        fpart = lane % P;
        const int fgrp = lane / P;
        fb = fgrp >> 2; fq = fgrp & 3;
        frow = warp * 4 + fq;
        act_k = (fq == 2 ? -2.0f : -1.0f) * 1.4426950408889634f;
        act_sc = fq == 2 ? 2.0f : 1.0f;
        act_of = fq == 2 ? -1.0f : 0.0f;
    }
};

// z_in: the input term of this lane's (batch row, gate) (projection output or bias); valid in lanes with fpart == 0.
// red_buf: partial sums of this pass, buffer already selected; NW warps wrote it.  nb: batch rows of this pass.
template <int NW>
__device__ __forceinline__ void finish_unit(const FinishLane &f, const float *red_buf, int RP, int WS, int nb, float z_in,
                                            float *c_unit /* [B] */, int b0, int B, int H, int j, unsigned stamp,
                                            unsigned long long *xch_parity /* [B][H] */, bool publish, float *y_row0, size_t y_bstride,
                                            __nv_bfloat16 *xb_row0, size_t xb_bstride, long long xb_plane, bool last_step,
                                            float *hT, float *cT)
{
    float z = 0.0f;
    if (f.fb < nb) {
        const float *rp = red_buf + f.fb * RP + f.frow;
        for (int w = f.fpart; w < NW; w += f.P) z += rp[(size_t)w * WS];
    }
    for (int o = f.P >> 1; o >= 1; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    z += z_in;
    const float act = gate_fast(z, f.act_k, f.act_sc, f.act_of);
    const int qb = f.fb * 4 * f.P;                 // lane of gate i of this batch row
    const float vi = __shfl_sync(0xffffffffu, act, qb);
    const float vf = __shfl_sync(0xffffffffu, act, qb + f.P);
    const float vg = __shfl_sync(0xffffffffu, act, qb + 2 * f.P);
    const float vo = __shfl_sync(0xffffffffu, act, qb + 3 * f.P);
    if (f.fq == 0 && f.fpart == 0 && f.fb < nb) {
        const int b = b0 + f.fb;
        const float cn = fmaf(vf, c_unit[b], vi * vg);
        const float hn = vo * tanh_fast(cn);
        if (publish)
            st_relaxed_u64(xch_parity + (size_t)b * H + j, ((unsigned long long)stamp << 32) | (unsigned long long)__float_as_uint(hn));
        c_unit[b] = cn;
        if (y_row0) y_row0[(size_t)b * y_bstride] = hn;
        if (xb_row0) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(hn);
            xb_row0[(size_t)b * xb_bstride] = hi;
            xb_row0[xb_plane + (size_t)b * xb_bstride] = __float2bfloat16_rn(hn - __bfloat162float(hi));
        }
        if (last_step) {
            if (hT) hT[(size_t)b * H + j] = hn;
            if (cT) cT[(size_t)b * H + j] = cn;
        }
    }
}


// ---------------------------------------------------------------------------------------------------
// Input projection inside a recurrent kernel's prologue (single sequence of at most kFuseMaxT steps): the CTA's
// own rows of G = X Wx^T + b for every timestep, left in shared memory as [kFuseMaxT][MT * 16 + 1] floats at
// byte offset gs_off.  Wx arrives as mma.sync operand-A fragments (xfrag_d: this direction's, laid out
// [cta][NW / 2 column ranges][nkx 16-column tiles][MT][32 lanes] uint4, the columns inside a tile permuted as
// described at the loads below); the activations are split into bf16 hi
// and lo terms on the fly.  Work split: the NW / 2 column ranges are each taken by two warps, one for the first
// 24 timesteps and one for the rest, so that the accumulators of a warp stay few and two loads can be in flight.
// Every warp leaves its partial products in its own block at the start of shared memory (NW * 24 * (MT * 16 + 1)
// floats, over memory the caller initialises only afterwards); then each (timestep, row) adds its NW / 2 partial
// sums in a fixed order and the bias.  All NW * 32 threads of the CTA call it; it ends with a CTA barrier.
template <int MT, int NW>
__device__ __forceinline__ float *fused_projection(unsigned char *smem, size_t gs_off, const float *X, const uint4 *xfrag_d,
                                                   const float *bias, int nkx, int in_l, int T, int H, int d, int cta,
                                                   int u0, int nu, int tid)
{
    constexpr int NT = NW * 32, NR = NW / 2, NTH = 3, GP = MT * 16 + 1;     // column ranges; 8-step tiles per warp
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tig = lane & 3;
    const int range = warp >> 1, half = warp & 1;
    const uint4 *xbase = xfrag_d + ((size_t)(cta * NR + range) * nkx) * MT * 32;
    for (int i = lane + 32 * half; i < nkx * MT * 4; i += 64)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(xbase) + (size_t)i * 128));
    float *G_s = nullptr;
    float pacc[MT][NTH][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTH; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) pacc[mt][nt][e] = 0.0f;
    const uint4 *xsrc = xbase + lane;
    const int t0 = half * NTH * 8;
    uint4 af[MT], an[MT];
    float xv[NTH][4], xn[NTH][4];
    const bool vec = (in_l & 3) == 0 && (reinterpret_cast<size_t>(X) & 15) == 0;     // rows of X start on 16 bytes
    auto fetch = [&](int i, uint4 (&fa)[MT], float (&fx)[NTH][4]) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) fa[mt] = i < nkx ? __ldg(xsrc + (size_t)(i * MT + mt) * 32) : make_uint4(0, 0, 0, 0);
        // The fragments are packed with the columns of a 16-wide tile permuted so that the four a lane multiplies
        // (MMA k slots 2 tig, 2 tig + 1, 2 tig + 8, 2 tig + 9) are the adjacent columns 4 tig .. 4 tig + 3: one
        // 16-byte load per (lane, timestep tile) where the rows of X allow it, four scalar loads otherwise.
        const int k0 = (range * nkx + i) * 16 + 4 * tig;
#pragma unroll
        for (int nt = 0; nt < NTH; ++nt) {
            const int t = t0 + nt * 8 + g;
            const float *xr = X + (size_t)t * in_l;
            if (vec && i < nkx && t < T && k0 + 3 < in_l) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(xr + k0));
                fx[nt][0] = v.x; fx[nt][1] = v.y; fx[nt][2] = v.z; fx[nt][3] = v.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) fx[nt][e] = (i < nkx && t < T && k0 + e < in_l) ? __ldg(xr + k0 + e) : 0.0f;
            }
        }
    };
    fetch(0, af, xv);
#pragma unroll 1
    for (int i = 0; i < nkx; ++i) {
        fetch(i + 1, an, xn);
#pragma unroll
        for (int nt = 0; nt < NTH; ++nt) {
            const __nv_bfloat162 h01 = __floats2bfloat162_rn(xv[nt][0], xv[nt][1]), h23 = __floats2bfloat162_rn(xv[nt][2], xv[nt][3]);
            const __nv_bfloat162 l01 = __floats2bfloat162_rn(xv[nt][0] - __low2float(h01), xv[nt][1] - __high2float(h01));
            const __nv_bfloat162 l23 = __floats2bfloat162_rn(xv[nt][2] - __low2float(h23), xv[nt][3] - __high2float(h23));
            const unsigned bh0 = *reinterpret_cast<const unsigned *>(&h01), bh1 = *reinterpret_cast<const unsigned *>(&h23);
            const unsigned bl0 = *reinterpret_cast<const unsigned *>(&l01), bl1 = *reinterpret_cast<const unsigned *>(&l23);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                mma_bf16(pacc[mt][nt], af[mt], bh0, bh1);
                mma_bf16(pacc[mt][nt], af[mt], bl0, bl1);
            }
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) af[mt] = an[mt];
#pragma unroll
        for (int nt = 0; nt < NTH; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) xv[nt][e] = xn[nt][e];
    }
    // every warp leaves its partial products in its own block (the blocks lie over shared memory that is only
    // initialised afterwards); then each (timestep, row) adds its NR partial sums in a fixed order and the bias
    constexpr int PP = MT * 16 + 1;
    float *P = reinterpret_cast<float *>(smem) + (size_t)warp * (NTH * 8) * PP;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTH; ++nt) {
            float *pp = P + (size_t)(nt * 8 + 2 * tig) * PP + mt * 16 + g;
            pp[0] = pacc[mt][nt][0];
            pp[PP] = pacc[mt][nt][1];
            pp[8] = pacc[mt][nt][2];
            pp[PP + 8] = pacc[mt][nt][3];
        }
    __syncthreads();
    G_s = reinterpret_cast<float *>(smem + gs_off);
    for (int i = tid; i < kFuseMaxT * MT * 16; i += NT) {
        const int t = i / (MT * 16), r = i - t * (MT * 16);
        const int hf = t / (NTH * 8), tl = t - hf * (NTH * 8);
        float sum = r < 4 * nu ? bias[(size_t)d * 4 * H + (size_t)u0 * 4 + r] : 0.0f;
#pragma unroll
        for (int rg = 0; rg < NR; ++rg) sum += reinterpret_cast<const float *>(smem)[((size_t)(2 * rg + hf) * (NTH * 8) + tl) * PP + r];
        G_s[(size_t)t * GP + r] = sum;
    }
    __syncthreads();
    return G_s;
}

}  // namespace lstm
