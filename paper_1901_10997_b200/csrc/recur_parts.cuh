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

}  // namespace lstm
