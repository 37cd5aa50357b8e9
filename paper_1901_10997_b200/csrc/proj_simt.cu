// Input staging and the CUDA-core forms of the input projection G = X Wx^T + b (the x_t half of
// W [x_t, h_{t-1}] + b in the paper's Section 4 cell equations, hoisted out of the time loop and
// computed for all timesteps at once).  The fp32 storage type uses the tiled FFMA kernel; pruned
// weights in CSR form use the sparse kernel.  The bf16 tensor-core kernel lives in proj_tc.cu.
#include "common.cuh"

namespace lstm {
namespace {

__global__ void stage_bf16_kernel(const float *__restrict__ x, __nv_bfloat16 *__restrict__ xb, long long plane,
                                  long long M, int K, int ld)
{
    const long long total = M * (long long)ld;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long m = i / ld;
        const int k = (int)(i - m * ld);
        const float v = k < K ? x[m * K + k] : 0.0f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        xb[i] = hi;
        xb[plane + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename WT> struct AccOf { typedef float T; };
template <> struct AccOf<float> { typedef double T; };   // fp32 storage accumulates in fp64

// 64x64 output tile, K step 16, 256 threads, 4x4 outputs per thread.
template <typename WT>
__global__ void __launch_bounds__(256) proj_simt_kernel(const float *__restrict__ X, const WT *__restrict__ W,
                                                        int ldw, const float *__restrict__ bias,
                                                        float *__restrict__ G, int M, int N, int K)
{
    __shared__ float xs[16][64 + 4];
    __shared__ float ws[16][64 + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int tm = (tid / 16) * 4, tn = (tid % 16) * 4;
    typedef typename AccOf<WT>::T AT;
    AT acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = (AT)0;

    for (int k0 = 0; k0 < K; k0 += 16) {
        // each thread loads 4 elements of each tile: row r = tid/4 (0..63), k = (tid%4)*4 .. +3
        const int r = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int k = k0 + kk + i;
            xs[kk + i][r] = (m0 + r < M && k < K) ? X[(size_t)(m0 + r) * K + k] : 0.0f;
            ws[kk + i][r] = (n0 + r < N && k < K) ? to_f32(W[(size_t)(n0 + r) * ldw + k]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float xv[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { xv[i] = xs[k][tm + i]; wv[i] = ws[k][tn + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma((AT)xv[i], (AT)wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + tm + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tn + j;
            if (n < N) G[(size_t)m * N + n] = (float)(acc[i][j] + (AT)(bias ? bias[n] : 0.0f));
        }
    }
}

// CSR projection: a CTA stages MT = 8 activation rows (transposed so that the 8 values of one column
// are contiguous) and its warps walk CSR rows; lanes stride over a row's entries.
constexpr int kCsrMT = 8;
constexpr int kCsrUnroll = 8;
template <typename AT>
__global__ void __launch_bounds__(256) proj_csr_kernel(const float *__restrict__ X, const int *__restrict__ rowptr,
                                                       const CsrEntry *__restrict__ ent,
                                                       const float *__restrict__ bias, float *__restrict__ G,
                                                       int M, int N, int K, int rows_per_cta)
{
    extern __shared__ __align__(16) float xt[];          // [K][8]
    const int m0 = blockIdx.y * kCsrMT;
    // a thread fetches one column of all eight rows at once (eight loads in flight, coalesced over the
    // threads) and stores them as the 32 contiguous bytes the row walk reads back
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        float v[kCsrMT];
#pragma unroll
        for (int mm = 0; mm < kCsrMT; ++mm) v[mm] = (m0 + mm < M) ? X[(size_t)(m0 + mm) * K + k] : 0.0f;
        *reinterpret_cast<float4 *>(xt + (size_t)k * kCsrMT) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4 *>(xt + (size_t)k * kCsrMT + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
    __syncthreads();
    // Rows are short (a few dozen to a few hundred survivors), so a warp walks four rows at once, eight
    // lanes each: four times as many independent trips to memory are in flight per warp, and the
    // reduction runs over eight lanes instead of thirty-two.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int sub = lane & 7, grp = lane >> 3;
    const int r_begin = blockIdx.x * rows_per_cta;
    const int r_end = min(N, r_begin + rows_per_cta);
    for (int rb = r_begin + warp * 4; rb < r_end; rb += nwarps * 4) {
        const int r = rb + grp;
        const bool live = r < r_end;
        AT acc[kCsrMT];
#pragma unroll
        for (int i = 0; i < kCsrMT; ++i) acc[i] = (AT)0;
        const int e_begin = live ? rowptr[r] : 0;
        const int e_end = live ? rowptr[r + 1] : 0;
        for (int e0 = e_begin + sub; e0 < e_end; e0 += 8 * kCsrUnroll) {
            CsrEntry en[kCsrUnroll];
#pragma unroll
            for (int u = 0; u < kCsrUnroll; ++u) {
                const int e = e0 + 8 * u;
                en[u] = e < e_end ? ent[e] : CsrEntry{0.0f, 0};
            }
#pragma unroll
            for (int u = 0; u < kCsrUnroll; ++u) {
                const float4 a = *reinterpret_cast<const float4 *>(xt + (size_t)en[u].col * kCsrMT);
                const float4 b = *reinterpret_cast<const float4 *>(xt + (size_t)en[u].col * kCsrMT + 4);
                const AT v = (AT)en[u].val;
                acc[0] = fma(v, (AT)a.x, acc[0]); acc[1] = fma(v, (AT)a.y, acc[1]);
                acc[2] = fma(v, (AT)a.z, acc[2]); acc[3] = fma(v, (AT)a.w, acc[3]);
                acc[4] = fma(v, (AT)b.x, acc[4]); acc[5] = fma(v, (AT)b.y, acc[5]);
                acc[6] = fma(v, (AT)b.z, acc[6]); acc[7] = fma(v, (AT)b.w, acc[7]);
            }
        }
#pragma unroll
        for (int i = 0; i < kCsrMT; ++i)
#pragma unroll
            for (int o = 4; o >= 1; o >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
        if (live && m0 + sub < M) {
            AT v = (AT)0;
#pragma unroll
            for (int i = 0; i < kCsrMT; ++i) v = (sub == i) ? acc[i] : v;
            G[(size_t)(m0 + sub) * N + r] = (float)(v + (AT)(bias ? bias[r] : 0.0f));
        }
    }
}

__global__ void proj_export_kernel(const float *__restrict__ G, int nsplit, long long split_stride,
                                   float *__restrict__ out, long long M, int D, int Hg)
{
    const long long total = M * D * 4 * Hg;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        // i enumerates the public layout [m][d][q][j]
        const int j = (int)(i % Hg);
        const int q = (int)((i / Hg) % 4);
        const long long md = i / (4 * Hg);
        const long long src = (md * Hg + j) * 4 + q;
        float v = 0.0f;
        for (int sp = 0; sp < nsplit; ++sp) v += G[sp * split_stride + src];
        out[i] = v;
    }
}

}  // namespace

cudaError_t launch_proj_export(const float *G, int nsplit, long long split_stride, float *out, long long M, int D, int Hg,
                               cudaStream_t st)
{
    const long long total = M * D * 4 * Hg;
    if (total == 0) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    proj_export_kernel<<<(int)blocks, 256, 0, st>>>(G, nsplit, split_stride, out, M, D, Hg);
    return cudaGetLastError();
}

cudaError_t launch_stage_bf16(const float *x, __nv_bfloat16 *xb, long long plane, long long M, int K, int ld,
                              cudaStream_t st)
{
    const long long total = M * (long long)ld;
    if (total == 0) return cudaSuccess;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 148LL * 8) blocks = 148LL * 8;
    stage_bf16_kernel<<<(int)blocks, threads, 0, st>>>(x, xb, plane, M, K, ld);
    return cudaGetLastError();
}

cudaError_t launch_proj_simt(const float *X, const void *W, bool bf16, int ldw, const float *bias,
                             float *G, int M, int N, int K, cudaStream_t st)
{
    if (M == 0 || N == 0) return cudaSuccess;
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    if (bf16)
        proj_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(X, (const __nv_bfloat16 *)W, ldw, bias, G, M, N, K);
    else
        proj_simt_kernel<float><<<grid, 256, 0, st>>>(X, (const float *)W, ldw, bias, G, M, N, K);
    return cudaGetLastError();
}

cudaError_t proj_csr_prepare(int max_smem)
{
    cudaError_t e = cudaFuncSetAttribute(proj_csr_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(proj_csr_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

cudaError_t launch_proj_csr(const float *X, const int *rowptr, const CsrEntry *ent, const float *bias,
                            float *G, int M, int N, int K, bool f64_acc, cudaStream_t st)
{
    if (M == 0 || N == 0) return cudaSuccess;
    const size_t smem = (size_t)K * kCsrMT * sizeof(float);
    const int mtiles = (M + kCsrMT - 1) / kCsrMT;
    int ctas_x = max(1, (148 * 4) / mtiles);      // about four CTAs per SM: a warp walks few rows, one trip to memory each
    int rows_per_cta = max(8, (N + ctas_x - 1) / ctas_x);
    ctas_x = (N + rows_per_cta - 1) / rows_per_cta;
    dim3 grid(ctas_x, mtiles);
    if (f64_acc) proj_csr_kernel<double><<<grid, 256, smem, st>>>(X, rowptr, ent, bias, G, M, N, K, rows_per_cta);
    else proj_csr_kernel<float><<<grid, 256, smem, st>>>(X, rowptr, ent, bias, G, M, N, K, rows_per_cta);
    return cudaGetLastError();
}

}  // namespace lstm
