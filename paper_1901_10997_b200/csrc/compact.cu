// Row/column-pruned stacks (paper, Section 4.2, Algorithm 1: whole rows and columns of the gate matrices are
// set to zero, which shrinks the model's dimension): the forward pass runs on an inner handle over the
// surviving hidden units only, and these two small kernels move states and outputs between the caller's full
// width and the compact one.
//
// A removed unit (all four gate rows zero in Wx and Wh, its column of Wh and of the next layer's Wx zero) is
// read by nobody and reads nothing: its gates are the constants i = sigmoid(b_i), f = sigmoid(b_f),
// g = tanh(b_g), o = sigmoid(b_o), so c_t = f c_{t-1} + i g and h_t = o tanh(c_t) follow from c_0 alone.  The
// scatter kernel evaluates that recurrence in fp64 for every removed unit and batch row (T dependent steps of
// a handful of operations each) beside copying the surviving units into place.
#include "common.cuh"

#include <algorithm>

namespace lstm {
namespace {

__global__ void compact_gather_kernel(CompactArgs a)
{
    const long long n = (long long)a.L * a.D * a.B * a.Hc;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int jc = (int)(i % a.Hc);
        const long long lb = i / a.Hc;                    // ld * B + b
        const int ld = (int)(lb / a.B);
        const long long src = lb * a.H + a.cmap[(size_t)ld * a.Hc + jc];
        if (a.h0 && a.h0c) a.h0c[i] = a.h0[src];
        if (a.c0 && a.c0c) a.c0c[i] = a.c0[src];
    }
}

__global__ void compact_scatter_kernel(CompactArgs a)
{
    const long long tid0 = blockIdx.x * (long long)blockDim.x + threadIdx.x, stride = (long long)gridDim.x * blockDim.x;
    // outputs of the last layer's surviving units
    const long long ny = (long long)a.T * a.B * a.D * a.Hc;
    for (long long i = tid0; i < ny; i += stride) {
        const int jc = (int)(i % a.Hc);
        const long long tbd = i / a.Hc;                   // (t * B + b) * D + d
        const int d = (int)(tbd % a.D);
        const int ld = (a.L - 1) * a.D + d;
        a.y[tbd * a.H + a.cmap[(size_t)ld * a.Hc + jc]] = a.yc[i];
    }
    // final states of every layer's surviving units
    const long long ns = (long long)a.L * a.D * a.B * a.Hc;
    for (long long i = tid0; i < ns; i += stride) {
        const int jc = (int)(i % a.Hc);
        const long long lb = i / a.Hc;
        const int ld = (int)(lb / a.B);
        const long long dst = lb * a.H + a.cmap[(size_t)ld * a.Hc + jc];
        if (a.hT) a.hT[dst] = a.hTc[i];
        if (a.cT) a.cT[dst] = a.cTc[i];
    }
    // removed units: the closed form, one thread per (removed unit, batch row)
    const long long nr = (long long)a.n_removed * a.B;
    for (long long i = tid0; i < nr; i += stride) {
        const int r = (int)(i / a.B), b = (int)(i % a.B);
        const int ld = a.rem_idx[2 * r], j = a.rem_idx[2 * r + 1];
        const int l = ld / a.D, d = ld % a.D;
        const double gi = 1.0 / (1.0 + exp(-(double)a.rem_bias[4 * r]));
        const double gf = 1.0 / (1.0 + exp(-(double)a.rem_bias[4 * r + 1]));
        const double gg = tanh((double)a.rem_bias[4 * r + 2]);
        const double go = 1.0 / (1.0 + exp(-(double)a.rem_bias[4 * r + 3]));
        const long long sidx = ((long long)ld * a.B + b) * a.H + j;
        double c = a.c0 ? (double)a.c0[sidx] : 0.0, h = 0.0;
        const bool last = l == a.L - 1;
        for (int s = 0; s < a.T; ++s) {
            c = gf * c + gi * gg;
            h = go * tanh(c);
            if (last) {
                const int t = d ? (a.T - 1 - s) : s;
                a.y[((long long)t * a.B + b) * a.D * a.H + (long long)d * a.H + j] = (float)h;
            }
        }
        if (a.hT) a.hT[sidx] = (float)h;
        if (a.cT) a.cT[sidx] = (float)c;
    }
}

}  // namespace

cudaError_t launch_compact_gather(const CompactArgs &a, cudaStream_t st)
{
    const long long n = (long long)a.L * a.D * a.B * a.Hc;
    if (n == 0) return cudaSuccess;
    compact_gather_kernel<<<(unsigned)std::min<long long>((n + 255) / 256, 592), 256, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_compact_scatter(const CompactArgs &a, cudaStream_t st)
{
    const long long n = std::max((long long)a.T * a.B * a.D * a.Hc, (long long)a.n_removed * a.B);
    if (n == 0) return cudaSuccess;
    compact_scatter_kernel<<<(unsigned)std::min<long long>((n + 255) / 256, 592), 256, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace lstm
