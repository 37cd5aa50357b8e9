// lstm_forward_noalloc: a one-layer, one-direction, fp32 LSTM forward pass for callers that must not
// allocate device memory.  Some callers of this library run where cudaMalloc is off limits: inside a
// latency-critical serving loop whose memory pool was carved up at start-up, under a framework's
// caching allocator that owns the whole device, or in a process that may not grow its footprint after
// initialisation.  lstm_create allocates (packed weights, workspace), so it is closed to them.  This
// entry point takes every tensor from the caller and keeps the only scratch it needs -- the per-step
// exchange words through which the CTAs of the persistent kernel hand h_t to each other, and a status
// word -- in a fixed array that is part of the library image.
//
// The kernel is a plain variant of the library's persistent recurrent kernel: weights stay in the
// caller's row-major fp32 arrays and are read through L2 each step (nothing is packed or made
// resident), the input half of the product is computed inside the step; sums and gate functions are
// evaluated in fp64 and stored as fp32, as in the handle's fp32 storage type.
#include "../../include/lstm_b200.h"

#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <mutex>

namespace {

constexpr int kMaxWords = LSTM_NOALLOC_MAX_BH;    // B * H exchange words per buffer
constexpr int kThreads = 256;
constexpr int kMaxDevices = 64;
constexpr long long kSpinLimit = 2000000000LL;     // clock64 ticks a wait may last (about a second)

struct Scratch {
    unsigned long long xch[2][kMaxWords];           // {step stamp : 32 | h bits : 32}, two step parities
    int status;
    int pad[63];
};

// Lives in the library image: every GPU that loads the library holds these 128.25 KiB until exit.
static __device__ __align__(256) unsigned char g_scratch[sizeof(Scratch)];

struct Args {
    const float *wx, *wh, *b, *x, *h0, *c0;
    float *y, *hT, *cT;
    int in_dim, H, T, B, ncta;
    int withhold_cta;           // failure-path self-test: this CTA never publishes its words (-1: none)
    long long spin_limit;       // clock64 ticks a wait may last
    Scratch *scratch;
};

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1) recur_noalloc_kernel(const Args a)
{
    extern __shared__ __align__(16) float smem[];
    __shared__ int abort_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
    const int H = a.H, in = a.in_dim, B = a.B, T = a.T;
    const int base = H / a.ncta, rem = H % a.ncta;
    const int c = blockIdx.x;
    const int nu = base + (c < rem ? 1 : 0);
    const int u0 = c * base + (c < rem ? c : rem);
    const int V = in + H;                              // one staged row: [x_t | h_{t-1}]
    float *v_s = smem;                                 // [B][V]
    float *c_s = smem + (size_t)B * V;                 // [upc][B]
    Scratch *sc = a.scratch;

    for (int i = tid; i < nu * B; i += kThreads) {
        const int u = i / B, bb = i - u * B;
        c_s[u * B + bb] = a.c0 ? a.c0[(size_t)bb * H + u0 + u] : 0.0f;
    }
    if (tid == 0) abort_s = 0;
    __syncthreads();

    for (int s = 0; s < T; ++s) {
        // ---- stage x_t and h_{t-1} of every batch row
        for (int i = tid; i < B * in; i += kThreads) {
            const int bb = i / in, k = i - bb * in;
            v_s[bb * V + k] = a.x[((size_t)s * B + bb) * in + k];
        }
        if (s == 0) {
            for (int i = tid; i < B * H; i += kThreads) {
                const int bb = i / H, k = i - bb * H;
                v_s[bb * V + in + k] = a.h0 ? a.h0[i] : 0.0f;
            }
        } else {
            const unsigned want = (unsigned)s;          // stamp of step s-1
            const unsigned long long *src = sc->xch[(s - 1) & 1];
            long long t_start = 0;
            for (int i = tid; i < B * H && !abort_s; i += kThreads) {
                unsigned long long w = ld_relaxed_u64(src + i);
                int rounds = 0;
                while ((unsigned)(w >> 32) != want) {
                    if ((++rounds & 63) == 0) {
                        const long long now = clock64();
                        if (t_start == 0) t_start = now;
                        if (now - t_start > a.spin_limit || *(volatile int *)&sc->status != 0) { abort_s = 1; break; }
                    }
                    w = ld_relaxed_u64(src + i);
                }
                const int bb = i / H, k = i - bb * H;
                v_s[bb * V + in + k] = __uint_as_float((unsigned)w);
            }
        }
        __syncthreads();
        if (abort_s) {
            if (tid == 0) atomicExch(&sc->status, LSTM_ERR_TIMEOUT);
            return;
        }
        // ---- one warp per (unit, batch row): four dot products over [x_t | h_{t-1}], gates, update
        for (int ub = warp; ub < nu * B; ub += nwarps) {
            const int u = ub / B, bb = ub - u * B;
            const int j = u0 + u;
            const float *v = v_s + (size_t)bb * V;
            // dot products and gate functions in fp64, like the handle's fp32 storage type: fp32 sums of a
            // few hundred terms already miss the 1e-4 agreement bound on outputs near zero
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float *rx = a.wx + (size_t)(q * H + j) * in;
                const float *rh = a.wh + (size_t)(q * H + j) * H;
                double sum = 0.0;
                for (int k = lane; k < in; k += 32) sum = fma((double)rx[k], (double)v[k], sum);
                for (int k = lane; k < H; k += 32) sum = fma((double)rh[k], (double)v[in + k], sum);
                acc[q] = sum;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], o);
            if (lane == 0) {
                const double zi = acc[0] + (a.b ? (double)a.b[j] : 0.0);
                const double zf = acc[1] + (a.b ? (double)a.b[H + j] : 0.0);
                const double zg = acc[2] + (a.b ? (double)a.b[2 * H + j] : 0.0);
                const double zo = acc[3] + (a.b ? (double)a.b[3 * H + j] : 0.0);
                const double gi = 1.0 / (1.0 + exp(-zi));
                const double gf = 1.0 / (1.0 + exp(-zf));
                const double gg = tanh(zg);
                const double go = 1.0 / (1.0 + exp(-zo));
                const double cn_d = fma(gf, (double)c_s[u * B + bb], gi * gg);
                const float cn = (float)cn_d;
                const float hn = (float)(go * tanh(cn_d));
                c_s[u * B + bb] = cn;
                if ((int)blockIdx.x != a.withhold_cta)
                st_relaxed_u64(&sc->xch[s & 1][(size_t)bb * H + j],
                               ((unsigned long long)(unsigned)(s + 1) << 32) | (unsigned long long)__float_as_uint(hn));
                a.y[((size_t)s * B + bb) * H + j] = hn;
                if (s == T - 1) {
                    if (a.hT) a.hT[(size_t)bb * H + j] = hn;
                    if (a.cT) a.cT[(size_t)bb * H + j] = cn;
                }
            }
        }
        __syncthreads();      // the staged rows are rewritten at the top of the next step
    }
}

// Per-device set-up record: the scratch array's device address (the symbol's name is only a host-side
// stand-in and must never be handed to a kernel), SM count, shared-memory limit.
struct DeviceSetup {
    bool ready = false;
    Scratch *scratch = nullptr;
    int sm_count = 0;
    int smem_optin = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

int fail(char *err, int errlen, int code, const char *fmt, ...)
{
    if (err && errlen > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(err, (size_t)errlen, fmt, ap);
        va_end(ap);
    }
    return code;
}

}  // namespace

extern "C" int lstm_forward_noalloc(const float *wx, const float *wh, const float *b, int in_dim, int hidden,
                                    const float *x, int T, int B, const float *h0, const float *c0,
                                    float *y, float *hT, float *cT, void *cuda_stream, char *err, int errlen)
{
    if (err && errlen > 0) err[0] = 0;
    if (in_dim < 1 || hidden < 1 || T < 0 || B < 0)
        return fail(err, errlen, LSTM_ERR_INVALID, "bad shape: in_dim=%d hidden=%d T=%d B=%d", in_dim, hidden, T, B);
    if ((long long)B * hidden > kMaxWords)
        return fail(err, errlen, LSTM_ERR_UNSUPPORTED,
                    "B*hidden = %lld exceeds the built-in scratch of %d exchange words (LSTM_NOALLOC_MAX_BH); "
                    "use lstm_create/lstm_forward for larger problems", (long long)B * hidden, kMaxWords);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t state_bytes = (size_t)B * hidden * sizeof(float);
    if (T == 0 || B == 0) {
        if (B > 0) {
            for (int i = 0; i < 2; ++i) {
                float *dst = i ? cT : hT;
                const float *src = i ? c0 : h0;
                if (!dst) continue;
                cudaError_t e = src ? cudaMemcpyAsync(dst, src, state_bytes, cudaMemcpyDeviceToDevice, st)
                                    : cudaMemsetAsync(dst, 0, state_bytes, st);
                if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "state copy failed: %s", cudaGetErrorString(e));
            }
        }
        return LSTM_OK;
    }
    if (!wx || !wh || !x || !y) return fail(err, errlen, LSTM_ERR_INVALID, "wx, wh, x and y must not be NULL");

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess)
        return fail(err, errlen, LSTM_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
    if (dev < 0 || dev >= kMaxDevices) return fail(err, errlen, LSTM_ERR_UNSUPPORTED, "device index %d not supported", dev);
    DeviceSetup ds;
    {
        // first call on this device: look up the scratch array's device address and the device limits
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        DeviceSetup &slot = g_setup[dev];
        if (!slot.ready) {
            int major = 0, coop = 0;
            cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&slot.sm_count, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&slot.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
            if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "device query failed: %s", cudaGetErrorString(e));
            if (major != 10 || !coop)
                return fail(err, errlen, LSTM_ERR_CUDA, "device is not an sm_100 GPU with cooperative launch");
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_scratch);
            if (e != cudaSuccess || !p)
                return fail(err, errlen, LSTM_ERR_CUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            e = cudaFuncSetAttribute(recur_noalloc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, slot.smem_optin - 1024);
            if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "kernel set-up failed: %s", cudaGetErrorString(e));
            slot.scratch = (Scratch *)p;
            slot.ready = true;
        }
        ds = slot;
    }

    Args a;
    a.wx = wx; a.wh = wh; a.b = b; a.x = x; a.h0 = h0; a.c0 = c0; a.y = y; a.hT = hT; a.cT = cT;
    a.in_dim = in_dim; a.H = hidden; a.T = T; a.B = B;
    a.ncta = hidden < ds.sm_count ? hidden : ds.sm_count;
    a.scratch = ds.scratch;
    a.withhold_cta = -1;
    a.spin_limit = kSpinLimit;
    // Failure-path self-test (see the header): LSTM_B200_NOALLOC_SELFTEST=<cta>:<clock ticks> makes that CTA withhold its
    // words, so the other CTAs' waits run out after the given ticks and the call returns LSTM_ERR_TIMEOUT.
    if (const char *env = getenv("LSTM_B200_NOALLOC_SELFTEST")) {
        int cta = -1; long long ticks = 0;
        if (sscanf(env, "%d:%lld", &cta, &ticks) == 2 && cta >= 0 && cta < a.ncta && ticks > 0) { a.withhold_cta = cta; a.spin_limit = ticks; }
    }
    const int upc = (hidden + a.ncta - 1) / a.ncta;
    const size_t smem = ((size_t)B * (in_dim + hidden) + (size_t)upc * B) * sizeof(float);
    if (smem > (size_t)ds.smem_optin - 1024)
        return fail(err, errlen, LSTM_ERR_UNSUPPORTED, "B*(in_dim+hidden) = %lld floats do not fit in shared memory",
                    (long long)B * (in_dim + hidden));

    // the array keeps the previous call's words: the stamps of this call restart at 1, so clear the part used
    cudaError_t e = cudaMemsetAsync(ds.scratch, 0, sizeof(Scratch), st);
    if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "scratch clear failed: %s", cudaGetErrorString(e));
    void *params[] = {&a};
    e = cudaLaunchCooperativeKernel((const void *)recur_noalloc_kernel, dim3(a.ncta), dim3(kThreads), params, smem, st);
    if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
    int status = 0;
    e = cudaMemcpyAsync(&status, &ds.scratch->status, sizeof status, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail(err, errlen, LSTM_ERR_CUDA, "run failed: %s", cudaGetErrorString(e));
    if (status != 0) return fail(err, errlen, status, "a device-side wait gave up (timeout); outputs are undefined");
    return LSTM_OK;
}
