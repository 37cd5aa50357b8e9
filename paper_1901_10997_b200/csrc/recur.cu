// Persistent recurrent kernel: the serial half of the LSTM forward pass (paper, Section 4, cell
// equations with zero hidden layers per gate):
//     z = G[t] + Wh h_{t-1};  i,f,o = sigmoid(z_i,z_f,z_o), g = tanh(z_g);  c_t = f c_{t-1} + i g;
//     h_t = o tanh(c_t)
// G[t] is the input projection (bias included) computed for all timesteps beforehand.
//
// Design.  One cooperative launch runs all T steps of one layer (both directions side by side on
// disjoint CTA groups).  Each CTA owns a contiguous range of hidden units and keeps the four gate rows
// of every owned unit resident in shared memory for the whole sequence (units that do not fit are
// streamed from L2 each step).  One warp computes the four dot products of a unit for a chunk of up to
// eight batch rows, reduces them with shuffles, applies the gate nonlinearities in four lanes at once
// and updates c and h.  The only cross-SM traffic per step is the exchange of h_t: each value is
// published as one 64-bit word {step stamp, value}; consumers poll the words themselves, so a step
// costs a single L2 round trip after the last producer's store and needs no separate barrier.
// Every wait is bounded: when it expires the CTA records a timeout status and leaves.
#include "common.cuh"
#include "device_util.cuh"

namespace lstm {
namespace {



__device__ __forceinline__ float sigmoid_f(float z) { return 1.0f / (1.0f + expf(-z)); }

// Position of hidden index k inside a staged h row.  Dense kernels read eight consecutive h values
// per lane as two 16-byte vectors; storing elements 0..3 and 4..7 of every group of eight in two
// separate planes keeps both vector reads free of bank conflicts.  The CSR kernel gathers single
// values and uses the identity layout.
template <bool PERM>
__device__ __forceinline__ int h_pos(int k, int Hs)
{
    if (PERM) return ((k >> 3) << 2) + (k & 3) + ((k & 4) ? (Hs >> 1) : 0);
    return k;
}

__device__ __forceinline__ float shfl_xor_at(float v, int o) { return __shfl_xor_sync(0xffffffffu, v, o); }
__device__ __forceinline__ double shfl_xor_at(double v, int o) { return __shfl_xor_sync(0xffffffffu, v, o); }
// arithmetic type of the gate functions and the state update, and the accumulator's value in it
template <typename AT> struct GateOf { typedef AT T; };
__device__ __forceinline__ float gate_value(float v) { return v; }
__device__ __forceinline__ double gate_value(double v) { return v; }

// Sum V values per lane over the 32 lanes of a warp.  On return lane l holds the total of value
// index l >> (5 - log2 V).  Each halving step exchanges half of the remaining values, so V values cost
// V - 1 + (5 - log2 V) shuffles instead of 5 V.
template <int V, typename AT>
__device__ __forceinline__ AT warp_reduce_multi(AT (&v)[V], int lane)
{
    constexpr int LOG2V = (V == 1) ? 0 : (V == 2) ? 1 : (V == 4) ? 2 : (V == 8) ? 3 : (V == 16) ? 4 : 5;
    static_assert((1 << LOG2V) == V, "V must be a power of two <= 32");
    int o = 16;
#pragma unroll
    for (int n = V; n > 1; n >>= 1) {
        const bool upper = (lane & o) != 0;
#pragma unroll
        for (int k = 0; k < n / 2; ++k) {
            const AT send = upper ? v[k] : v[k + n / 2];
            const AT keep = upper ? v[k + n / 2] : v[k];
            v[k] = keep + shfl_xor_at(send, o);
        }
        o >>= 1;
    }
#pragma unroll
    for (int o2 = (16 >> LOG2V); o2 >= 1; o2 >>= 1) v[0] += shfl_xor_at(v[0], o2);
    return v[0];
}


// eight weights of one row at vector index v8 -> fp32
__device__ __forceinline__ void load_w8(const __nv_bfloat16 *row, int v8, float (&w)[8])
{
    const uint4 p = *reinterpret_cast<const uint4 *>(row + (size_t)v8 * 8);
    const unsigned x[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[2 * i] = __uint_as_float(x[i] << 16);
        w[2 * i + 1] = __uint_as_float(x[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void load_w8(const float *row, int v8, float (&w)[8])
{
    const float4 a = *reinterpret_cast<const float4 *>(row + (size_t)v8 * 8);
    const float4 b = *reinterpret_cast<const float4 *>(row + (size_t)v8 * 8 + 4);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}

// Dense: four gate rows of one unit times BT staged h rows.  rows points at [4][Hp8] weights in
// shared or global memory (the caller picks; the branch is warp-uniform).
template <typename WT, int BT, typename AT>
__device__ __forceinline__ void unit_dot_dense(const WT *rows, int Hp8, const float *hb, int Hs,
                                               int lane, AT (&acc)[4 * BT])
{
    const int nv = Hp8 >> 3;
    for (int v8 = lane; v8 < nv; v8 += 32) {
        float4 hlo[BT], hhi[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            hlo[b] = *reinterpret_cast<const float4 *>(hb + b * Hs + v8 * 4);
            hhi[b] = *reinterpret_cast<const float4 *>(hb + b * Hs + (Hs >> 1) + v8 * 4);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float w[8];
            load_w8(rows + (size_t)q * Hp8, v8, w);
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                AT s = acc[q * BT + b];
                s = fma((AT)w[0], (AT)hlo[b].x, s); s = fma((AT)w[1], (AT)hlo[b].y, s);
                s = fma((AT)w[2], (AT)hlo[b].z, s); s = fma((AT)w[3], (AT)hlo[b].w, s);
                s = fma((AT)w[4], (AT)hhi[b].x, s); s = fma((AT)w[5], (AT)hhi[b].y, s);
                s = fma((AT)w[6], (AT)hhi[b].z, s); s = fma((AT)w[7], (AT)hhi[b].w, s);
                acc[q * BT + b] = s;
            }
        }
    }
}

// CSR entry decoding: bf16 entries are one 32-bit word {col:16 | bf16 value:16}; fp32 entries are
// {value, col} pairs.  Rows are padded to a multiple of four entries (value 0, column 0).
struct EntBf16 { typedef uint4 vec4; };
__device__ __forceinline__ void decode4(const unsigned *ent, int vi, float (&w)[4], int (&col)[4])
{
    const uint4 p = *reinterpret_cast<const uint4 *>(ent + (size_t)vi * 4);
    const unsigned x[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { w[i] = __uint_as_float(x[i] << 16); col[i] = (int)(x[i] >> 16); }
}
__device__ __forceinline__ void decode4(const CsrEntry *ent, int vi, float (&w)[4], int (&col)[4])
{
    const uint4 p0 = *reinterpret_cast<const uint4 *>(ent + (size_t)vi * 4);
    const uint4 p1 = *reinterpret_cast<const uint4 *>(ent + (size_t)vi * 4 + 2);
    w[0] = __uint_as_float(p0.x); col[0] = (int)p0.y; w[1] = __uint_as_float(p0.z); col[1] = (int)p0.w;
    w[2] = __uint_as_float(p1.x); col[2] = (int)p1.y; w[3] = __uint_as_float(p1.z); col[3] = (int)p1.w;
}

// CSR: the four gate rows of a unit are consecutive rows; e[0..4] are their entry offsets relative to
// `ent` (multiples of 4).  Each lane takes whole 4-entry vectors, so a vector never straddles rows.
template <typename ET, int BT, typename AT>
__device__ __forceinline__ void unit_dot_csr(const ET *ent, const int (&e)[5], const float *hb, int Hs,
                                             int lane, AT (&acc)[4 * BT])
{
    for (int vi = (e[0] >> 2) + lane; vi < (e[4] >> 2); vi += 32) {
        const int pos = vi << 2;
        const int q = (pos >= e[1]) + (pos >= e[2]) + (pos >= e[3]);
        float w[4]; int col[4];
        decode4(ent, vi, w, col);
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            AT s = (AT)w[0] * (AT)hb[b * Hs + col[0]];
            s = fma((AT)w[1], (AT)hb[b * Hs + col[1]], s);
            s = fma((AT)w[2], (AT)hb[b * Hs + col[2]], s);
            s = fma((AT)w[3], (AT)hb[b * Hs + col[3]], s);
#pragma unroll
            for (int qq = 0; qq < 4; ++qq) acc[qq * BT + b] += (q == qq) ? s : (AT)0;
        }
    }
}

// bf16 storage: fp32 accumulation and gate functions.  fp32 storage: dot products accumulate in fp64
// and the gate functions are evaluated in fp64, so the only fp32 roundings left are the stored
// projection, h and c -- what the 1e-4 agreement bound of that mode needs.  Cheaper forms were measured
// and miss it: fp32 chains of eight terms summed in fp64 (1.2e-4 on the floored metric at H = 300, B = 16),
// two-float sums with fp32 gate functions (1.02e-4); neither shortened the step, which waits for the exchange.
template <bool BF16> struct Types { typedef __nv_bfloat16 W; typedef unsigned E; typedef float A; };
template <> struct Types<false> { typedef float W; typedef CsrEntry E; typedef double A; };

__device__ __forceinline__ float gate_fn(float z, bool is_tanh) { return is_tanh ? tanhf(z) : sigmoid_f(z); }
__device__ __forceinline__ double gate_fn(double z, bool is_tanh) { return is_tanh ? tanh(z) : 1.0 / (1.0 + exp(-z)); }
__device__ __forceinline__ float tanh_t(float c) { return tanhf(c); }
__device__ __forceinline__ double tanh_t(double c) { return tanh(c); }

// ONE: a single sequence (B = 1, BT = 1): the batch-row arithmetic folds away at compile time.
template <bool BF16, int BT, bool CSR, bool ONE = false>
__global__ void __launch_bounds__(512, 1) recur_kernel(const RecurArgs a)
{
    typedef typename Types<BF16>::W WT;
    typedef typename Types<BF16>::E ET;
    typedef typename Types<BF16>::A AT;
    constexpr int V = 4 * BT;
    constexpr int SH = (V == 4) ? 3 : (V == 8) ? 2 : (V == 16) ? 1 : 0;   // lane -> value index shift

    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int abort_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int H = a.H, Hs = a.Hs, B = ONE ? 1 : a.B, T = a.T, D = a.D;
    const int d = a.dir0 + blockIdx.x / a.ncta_dir;
    const int cta = blockIdx.x % a.ncta_dir;
    int u0, nu;
    unit_range(H, a.ncta_dir, cta, u0, nu);
    const int upc = (H + a.ncta_dir - 1) / a.ncta_dir;

    // shared-memory carve-up: staged h (two buffers of BT rows), c state, resident weights
    // (stage_all: two buffers of all B rows, so that a step polls its exchange words in one phase)
    // (rounded up to whole chunks: the products of the last chunk read BT rows, the ones beyond B stay zero)
    const int rows_staged = a.stage_all ? ((B + BT - 1) / BT) * BT : BT;
    float *h_s = reinterpret_cast<float *>(smem);
    float *c_s = h_s + 2 * rows_staged * Hs;
    unsigned char *w_s = reinterpret_cast<unsigned char *>(c_s + ((upc * B + 3) & ~3));
    LSTM_CHECK_SMEM_END((size_t)(w_s - smem) + (size_t)a.w_smem_bytes, a.status);

    // ---- residency: how many leading units of this CTA live in shared memory
    int units_res = 0;
    const WT *wg = nullptr;        // dense: this CTA's [nu][4][Hp8] block in global memory
    const ET *eg = nullptr;        // CSR: entries of this direction in global memory
    const int *rp_s = nullptr;     // CSR: row offsets of this CTA's rows (4 nu + 1), in shared memory
    int ent_base = 0;              // CSR: first entry of this CTA's slice
    if (!CSR) {
        const size_t unit_bytes = (size_t)4 * a.Hp8 * sizeof(WT);
        wg = reinterpret_cast<const WT *>(a.wh[d]) + (size_t)u0 * 4 * a.Hp8;
        units_res = (int)min((size_t)nu, (size_t)a.w_smem_bytes / unit_bytes);
        const uint4 *src = reinterpret_cast<const uint4 *>(wg);
        uint4 *dst = reinterpret_cast<uint4 *>(w_s);
        const int n16 = (int)((size_t)units_res * unit_bytes / 16);
        for (int i = tid; i < n16; i += nthreads) dst[i] = __ldg(src + i);
    } else {
        // layout: [4 upc + 1 row offsets, padded to 4 ints][entries...]
        int *rp = reinterpret_cast<int *>(w_s);
        const int *gp = a.csr_ptr[d] + (size_t)u0 * 4;
        for (int i = tid; i <= 4 * nu; i += nthreads) rp[i] = gp[i];
        rp_s = rp;
        eg = reinterpret_cast<const ET *>(a.csr_ent[d]);
        __syncthreads();
        ent_base = rp[0];
        const int rp_bytes = ((4 * upc + 1 + 3) & ~3) * 4;
        const long long room = ((long long)a.w_smem_bytes - rp_bytes) / (long long)sizeof(ET);
        while (units_res < nu && (long long)(rp[4 * (units_res + 1)] - ent_base) <= room) ++units_res;
        const int nent = rp[4 * units_res] - ent_base;                       // multiple of 4
        const uint4 *src = reinterpret_cast<const uint4 *>(eg + ent_base);
        uint4 *dst = reinterpret_cast<uint4 *>(w_s + rp_bytes);
        const int n16 = (int)((size_t)nent * sizeof(ET) / 16);
        for (int i = tid; i < n16; i += nthreads) dst[i] = __ldg(src + i);
    }
    const unsigned char *res_base = CSR ? w_s + ((4 * upc + 1 + 3) & ~3) * 4 : w_s;

    for (int i = tid; i < 2 * rows_staged * Hs; i += nthreads) h_s[i] = 0.0f;
    for (int i = tid; i < nu * B; i += nthreads) {
        const int u = i / B, b = i - u * B;
        c_s[u * B + b] = a.c0 ? a.c0[((size_t)d * B + b) * H + u0 + u] : 0.0f;
    }
    if (tid == 0) abort_s = 0;
    __syncthreads();

    const int nchunk = (B + BT - 1) / BT;
    unsigned long long *xch_d = a.xch + (size_t)d * 2 * B * H;
    const int vidx = lane >> SH;            // value index this lane holds after the reduction
    const int q_mine = vidx / BT;           // its gate
    const int b_mine = vidx % BT;           // its batch row inside the chunk
    const int b_gather = lane & (BT - 1);   // batch row a lane < BT finalises

    // gates and state update of unit u for the batch rows b0 .. b0+nb-1 staged at hb; g_pl: the projection terms
    // fetched ahead for this lane (valid when g_ahead), else they are loaded here
    auto process_unit = [&](int u, int b0, int nb, const float *hb, bool g_ahead, const float (&g_pl)[4], int s, int t) {
        AT acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = (AT)0;
        if (!CSR) {
            // one copy of the loop serves resident (shared) and streamed (global) units: the
            // base pointer is warp-uniform and the loads are generic
            const WT *rows = (u < units_res) ? reinterpret_cast<const WT *>(res_base) + (size_t)u * 4 * a.Hp8
                                             : wg + (size_t)u * 4 * a.Hp8;
            unit_dot_dense<WT, BT, AT>(rows, a.Hp8, hb, Hs, lane, acc);
        } else {
            int e[5];
#pragma unroll
            for (int i = 0; i < 5; ++i) e[i] = rp_s[4 * u + i] - ent_base;
            const ET *ents = (u < units_res) ? reinterpret_cast<const ET *>(res_base) : eg + ent_base;
            unit_dot_csr<ET, BT, AT>(ents, e, hb, Hs, lane, acc);
        }
        AT z = warp_reduce_multi<V, AT>(acc, lane);

        float g_in = (g_pl[0] + g_pl[1]) + (g_pl[2] + g_pl[3]);
        if (!g_ahead) {
            g_in = 0.0f;
            if (b_mine < nb) {
                const float *gp = a.G + (((size_t)t * B + b0 + b_mine) * D + d) * 4 * H +
                                  (size_t)(u0 + u) * 4 + q_mine;
                for (int sp = 0; sp < a.nsplit; ++sp)
                    g_in += __ldg(gp + (size_t)sp * a.g_split_stride);
            }
        }
        z += (AT)g_in;
        typedef typename GateOf<AT>::T GT;
        const GT act = gate_fn(gate_value(z), q_mine == 2);
        const GT vi = __shfl_sync(0xffffffffu, act, (0 * BT + b_gather) << SH);
        const GT vf = __shfl_sync(0xffffffffu, act, (1 * BT + b_gather) << SH);
        const GT vg = __shfl_sync(0xffffffffu, act, (2 * BT + b_gather) << SH);
        const GT vo = __shfl_sync(0xffffffffu, act, (3 * BT + b_gather) << SH);
        if (lane < nb) {
            const int b = b0 + lane;
            const int j = u0 + u;
            const GT cn_a = fma(vf, (GT)c_s[u * B + b], vi * vg);
            const float cn = (float)cn_a;
            const float hn = (float)(vo * tanh_t(cn_a));
            if ((int)blockIdx.x != a.withhold_cta)
            st_relaxed_u64(xch_d + ((size_t)(s & 1) * B + b) * H + j,
                           ((unsigned long long)(a.stamp_base + (unsigned)s + 1u) << 32) |
                               (unsigned long long)__float_as_uint(hn));
            c_s[u * B + b] = cn;
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
    };

#pragma unroll 1
    for (int s = 0; s < T; ++s) {
        const int t = d ? (T - 1 - s) : s;
        if (a.stage_all) {
            // ---- all B rows of h_{t-1} in ONE polling phase (eight words per thread in flight over the flattened
            // [B][H] block), then every (unit, chunk of BT rows) pair on its own warp
            float *buf = h_s + (size_t)(s & 1) * rows_staged * Hs;
            const int total = B * H;
            // projection terms of this warp's first (unit, chunk) item, requested before the wait
            float g_first[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (warp < nu * nchunk) {
                const int u = warp / nchunk, b0 = (warp - u * nchunk) * BT;
                if (b0 + b_mine < B) {
                    const float *gp = a.G + (((size_t)t * B + b0 + b_mine) * D + d) * 4 * H + (size_t)(u0 + u) * 4 + q_mine;
#pragma unroll
                    for (int sp = 0; sp < 4; ++sp)
                        if (sp < a.nsplit) g_first[sp] = ld_nc_early(gp + (size_t)sp * a.g_split_stride);
                }
            }
            if (s == 0) {
                for (int i = tid; i < total; i += nthreads) {
                    const int b = i / H, k = i - b * H;
                    buf[b * Hs + h_pos<!CSR>(k, Hs)] = a.h0 ? a.h0[(size_t)d * B * H + i] : 0.0f;
                }
            } else {
                const unsigned want = a.stamp_base + (unsigned)s;
                const unsigned long long *src = xch_d + (size_t)((s - 1) & 1) * B * H;
                long long t_start = 0;
                bool gave_up = false;
                for (int base = tid; base < total && !gave_up; base += 8 * nthreads) {
                    unsigned pending = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) pending |= (base + i * nthreads < total) ? (1u << i) : 0u;
                    int rounds = 0;
                    while (pending) {
                        unsigned long long w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (pending & (1u << i)) w[i] = ld_relaxed_u64(src + base + i * nthreads);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if ((pending & (1u << i)) && (unsigned)(w[i] >> 32) == want) {
                                const int idx = base + i * nthreads, b = idx / H, k = idx - b * H;
                                buf[b * Hs + h_pos<!CSR>(k, Hs)] = __uint_as_float((unsigned)w[i]);
                                pending &= ~(1u << i);
                            }
                        if (pending && ((++rounds & 63) == 0)) {
                            const long long now = clock64();
                            if (t_start == 0) t_start = now;
                            if (now - t_start > a.spin_limit || ld_volatile_s32(a.status) != kStatusOk) {
                                gave_up = true;
                                break;
                            }
                        }
                    }
                }
                if (gave_up) abort_s = 1;
            }
            __syncthreads();
            if (abort_s) {
                if (tid == 0) atomicExch(a.status, kStatusTimeout);
                return;
            }
            const float no_g[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 1
            for (int item = warp; item < nu * nchunk; item += nwarps) {
                const int u = item / nchunk, ci = item - u * nchunk, b0 = ci * BT;
                if (item == warp) process_unit(u, b0, min(BT, B - b0), buf + (size_t)b0 * Hs, true, g_first, s, t);
                else process_unit(u, b0, min(BT, B - b0), buf + (size_t)b0 * Hs, false, no_g, s, t);
            }
            __syncthreads();        // pacing, as below: polls only after this CTA's own stores
            continue;
        }
#pragma unroll 1
        for (int ci = 0; ci < nchunk; ++ci) {
            const int b0 = ci * BT;
            const int nb = min(BT, B - b0);
            float *hb = h_s + (size_t)((s * nchunk + ci) & 1) * BT * Hs;

            // projection term of this warp's first unit, fetched before the wait
            // (one register per split-K plane, added up only after the wait, so the loads stay in flight)
            float g_pl[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (warp < nu && b_mine < nb) {
                const float *gp = a.G + (((size_t)t * B + b0 + b_mine) * D + d) * 4 * H +
                                  (size_t)(u0 + warp) * 4 + q_mine;
#pragma unroll
                for (int sp = 0; sp < 4; ++sp)
                    if (sp < a.nsplit) g_pl[sp] = ld_nc_early(gp + (size_t)sp * a.g_split_stride);
            }

            // ---- stage h_{t-1} rows b0 .. b0+nb-1 into shared memory
            if (s == 0) {
                for (int b = 0; b < nb; ++b)
                    for (int k = tid; k < H; k += nthreads)
                        hb[b * Hs + h_pos<!CSR>(k, Hs)] =
                            a.h0 ? a.h0[((size_t)d * B + b0 + b) * H + k] : 0.0f;
            } else {
                const unsigned want = a.stamp_base + (unsigned)s;      // stamp of step s-1
                const unsigned long long *src = xch_d + ((size_t)((s - 1) & 1) * B + b0) * H;
                long long t_start = 0;
                bool gave_up = false;
                for (int b = 0; b < nb && !gave_up; ++b) {
                    const unsigned long long *row = src + (size_t)b * H;
                    float *hrow = hb + b * Hs;
                    for (int kb = tid; kb < H && !gave_up; kb += 8 * nthreads) {
                        unsigned pending = 0;
#pragma unroll
                        for (int i = 0; i < 8; ++i) pending |= (kb + i * nthreads < H) ? (1u << i) : 0u;
                        int rounds = 0;
                        while (pending) {
                            unsigned long long w[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if (pending & (1u << i)) w[i] = ld_relaxed_u64(row + kb + i * nthreads);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if ((pending & (1u << i)) && (unsigned)(w[i] >> 32) == want) {
                                    hrow[h_pos<!CSR>(kb + i * nthreads, Hs)] = __uint_as_float((unsigned)w[i]);
                                    pending &= ~(1u << i);
                                }
                            if (pending && ((++rounds & 63) == 0)) {
                                const long long now = clock64();
                                if (t_start == 0) t_start = now;
                                if (now - t_start > a.spin_limit || ld_volatile_s32(a.status) != kStatusOk) {
                                    gave_up = true;
                                    break;
                                }
                            }
                        }
                    }
                }
                if (gave_up) abort_s = 1;
            }
            __syncthreads();
            if (abort_s) {
                if (tid == 0) atomicExch(a.status, kStatusTimeout);
                return;
            }

            // ---- gates and state update, one unit per warp at a time
#pragma unroll 1
            for (int u = warp; u < nu; u += nwarps) process_unit(u, b0, nb, hb, u == warp, g_pl, s, t);
            // Pacing: no warp starts to poll for the next pass before this CTA has issued its own stores;
            // loads that spin on words that are not there yet would sit in front of those stores on the
            // way to L2 and delay every other CTA.
            __syncthreads();
        }
    }
}

template <bool BF16, bool CSR>
cudaError_t launch_bt(const RecurArgs &a, int threads, size_t smem, cudaStream_t st)
{
    const void *fn = nullptr;
    switch (a.BT) {
        case 1: fn = a.B == 1 ? (const void *)recur_kernel<BF16, 1, CSR, true> : (const void *)recur_kernel<BF16, 1, CSR>; break;
        case 2: fn = (const void *)recur_kernel<BF16, 2, CSR>; break;
        case 4: fn = (const void *)recur_kernel<BF16, 4, CSR>; break;
        case 8: fn = (const void *)recur_kernel<BF16, 8, CSR>; break;
        default: return cudaErrorInvalidValue;
    }
    RecurArgs copy = a;
    void *params[] = {&copy};
    return cudaLaunchCooperativeKernel(fn, dim3(a.ncta_dir * (a.ndirs ? a.ndirs : a.D)), dim3(threads), params, smem, st);
}

template <bool BF16, bool CSR>
cudaError_t prepare_all(int max_smem)
{
    cudaError_t e;
    e = cudaFuncSetAttribute(recur_kernel<BF16, 1, CSR>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(recur_kernel<BF16, 1, CSR, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(recur_kernel<BF16, 2, CSR>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(recur_kernel<BF16, 4, CSR>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(recur_kernel<BF16, 8, CSR>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

}  // namespace

cudaError_t launch_recur_dense(const RecurArgs &a, bool bf16, int threads, size_t smem, cudaStream_t st)
{
    return bf16 ? launch_bt<true, false>(a, threads, smem, st) : launch_bt<false, false>(a, threads, smem, st);
}
cudaError_t launch_recur_csr(const RecurArgs &a, bool bf16, int threads, size_t smem, cudaStream_t st)
{
    return bf16 ? launch_bt<true, true>(a, threads, smem, st) : launch_bt<false, true>(a, threads, smem, st);
}
cudaError_t recur_dense_prepare(int max_smem)
{
    cudaError_t e = prepare_all<true, false>(max_smem);
    return e != cudaSuccess ? e : prepare_all<false, false>(max_smem);
}
cudaError_t recur_csr_prepare(int max_smem)
{
    cudaError_t e = prepare_all<true, true>(max_smem);
    return e != cudaSuccess ? e : prepare_all<false, true>(max_smem);
}

}  // namespace lstm
