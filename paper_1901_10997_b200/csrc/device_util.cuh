// Device-side helpers shared by the kernels of the lstm_b200 library: the stamped-word exchange
// primitives, named barriers, the warp-level tensor instruction, the gate functions, and the
// mbarrier / TMA / tcgen05 wrappers of the two tensor-core kernels, plus the host-side tensor-map
// encoder.  One definition each, so that a fix to a descriptor or a fence is made once.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace lstm {

// ---------------------------------------------------------------------------------------------------
// Checked build (-DLSTM_B200_CHECKED): the stand-in for a memory checker.  Index and carve-up checks compile
// into the kernels; a violation records kStatusInternal in the status word (reported as LSTM_ERR_INTERNAL) and
// the access is skipped -- nothing traps, nothing reads or writes out of range.  In the normal build the macros
// vanish.
// ---------------------------------------------------------------------------------------------------
constexpr int kStatusInternal = 6;
__device__ __forceinline__ unsigned dynamic_smem_bytes()
{
    unsigned v;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(v));
    return v;
}
#ifdef LSTM_B200_CHECKED
__device__ __forceinline__ bool check_index(long long i, long long n, int *status)
{
    if (i >= 0 && i < n) return true;
    atomicCAS(status, 0, kStatusInternal);
    return false;
}
#define LSTM_CHECK_INDEX(i, n, status) lstm::check_index((long long)(i), (long long)(n), (status))
// end_bytes: bytes of dynamic shared memory the kernel is about to carve up (or read as an operand)
#define LSTM_CHECK_SMEM_END(end_bytes, status) \
    do { if ((unsigned long long)(end_bytes) > (unsigned long long)lstm::dynamic_smem_bytes()) atomicCAS((status), 0, lstm::kStatusInternal); } while (0)
#else
#define LSTM_CHECK_INDEX(i, n, status) true
#define LSTM_CHECK_SMEM_END(end_bytes, status) do { } while (0)
#endif

// ---------------------------------------------------------------------------------------------------
// global-memory accesses of the exchange
// ---------------------------------------------------------------------------------------------------
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
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u32(unsigned *p, unsigned v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// release store at GPU scope: what this thread wrote, and what it observed others write (a CTA barrier counts),
// is visible to whoever reads the value with acquire semantics or fences after reading it
__device__ __forceinline__ void st_release_u32(unsigned *p, unsigned v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_volatile_s32(const int *p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// read-only loads that the compiler may not sink towards their use: issued early, consumed a step later
__device__ __forceinline__ float ld_nc_early(const float *p)
{
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_nc_f4(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
// release / acquire fence at GPU scope (lighter than the sequentially consistent __threadfence)
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

// 16-byte asynchronous copy global -> shared through L2 only (never a stale L1 line)
__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// named barriers over n threads of the CTA
__device__ __forceinline__ void bar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void bar_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// D += A (16x16, row) * B (16x8, col), bf16 inputs, fp32 accumulation
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4 &a, unsigned b0, unsigned b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// ---------------------------------------------------------------------------------------------------
// Gate functions from the fast exponential: absolute error of a few 1e-7, far inside the 2e-2 bound of the
// bf16 storage type.  Both are one expression, sc / (1 + 2^(-k log2(e) z)) + of: the logistic function with
// (k, sc, of) = (1, 1, 0) and tanh z = 2 logistic(2z) - 1 with (2, 2, -1): one exponential and one
// reciprocal on the path from the summed pre-activation to the published h.
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float gate_fast(float z, float neg_k_log2e, float sc, float of)
{
    return fmaf(sc, __fdividef(1.0f, 1.0f + ex2_fast(neg_k_log2e * z)), of);
}
__device__ __forceinline__ float sigmoid_fast(float z) { return __fdividef(1.0f, 1.0f + ex2_fast(-1.4426950408889634f * z)); }
__device__ __forceinline__ float tanh_fast(float z) { return fmaf(2.0f, __fdividef(1.0f, 1.0f + ex2_fast(-2.8853900817779268f * z)), -1.0f); }

// hidden units [u0, u0 + n) of CTA c when H units are split evenly over nc CTAs
__host__ __device__ __forceinline__ void unit_range(int H, int nc, int c, int &u0, int &n)
{
    const int base = H / nc, rem = H % nc;
    n = base + (c < rem ? 1 : 0);
    u0 = c * base + (c < rem ? c : rem);
}

// ---------------------------------------------------------------------------------------------------
// mbarrier, TMA and tcgen05 wrappers
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
constexpr long long kMbarWaitTicks = 4000000000ll;   // clock64 ticks an mbarrier wait may last (about two seconds)
// Bounded wait.  Returns false when it gave up (or another role did): the caller leaves its loop.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    long long t_start = 0;
    for (long long it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255) == 255) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t_start == 0) t_start = now;
            if (now - t_start > kMbarWaitTicks) break;
        }
    }
    *abort_flag = 1;
    return false;
}
// tiled TMA load of one box into this CTA's shared memory (no multicast: every CTA fetches its own tiles)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// K-major operand tile in shared memory, 128-byte swizzle: rows of 128 bytes, groups of 8 rows are
// 1024 bytes apart (stride byte offset); version field = 1 for this architecture.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);          // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                                 // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                       // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                                 // descriptor version
    d |= (uint64_t)2 << 61;                                 // layout type: 128-byte swizzle
    return d;
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}

// ---------------------------------------------------------------------------------------------------
// Host: tensor map of a row-major bf16 matrix [rows][ld] of which `cols` columns are valid, boxes of
// box_rows x 64 columns, 128-byte swizzle, zero fill outside.  The driver entry point is looked up through
// the runtime, so the library links against the runtime only.
// ---------------------------------------------------------------------------------------------------
inline bool encode_tmap_bf16_2d(void *map128, const void *base, long long rows, long long cols, long long ld, int box_rows)
{
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return false;
        fn = (EncodeFn)p;
    }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    return fn((CUtensorMap *)map128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace lstm
