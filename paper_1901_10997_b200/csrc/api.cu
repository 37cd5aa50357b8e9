// C ABI of the lstm_b200 library: create-time packing, the per-layer launch sequence, host-buffer
// variant, status and measurement support.  See include/lstm_b200.h for the contract.
#include "../../include/lstm_b200.h"
#include "common.cuh"
#include "csr_pack.h"
#include "device_util.cuh"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace lstm;

namespace {

thread_local std::string g_create_error;

struct Layer {
    int in_l = 0;
    int ldk = 0;                       // row stride of wx (elements)
    void *wx = nullptr;                // dense [D*4H][ldk], rows in order d*4H + j*4 + q
    float *bias = nullptr;             // [D*4H], same order
    int *wx_rowptr = nullptr;          // CSR projection [D*4H + 1]
    CsrEntry *wx_ent = nullptr;
    void *wh[2] = {nullptr, nullptr};  // dense [H][4][Hp8]
    int *wh_ptr[2] = {nullptr, nullptr};   // CSR recurrence: padded entry offsets [4H+1]
    void *wh_ent[2] = {nullptr, nullptr};
    uint4 *wfrag[2] = {nullptr, nullptr};  // register-resident kernel: operand-A fragments
    uint4 *xfrag[2] = {nullptr, nullptr};  //   and Wx in the same layout (projection fused into the kernel's prologue)
    int nkw_x = 0;
    __nv_bfloat16 *wtc = nullptr;          // batched tensor-core kernel: [D * ncta * RA][ld64] rows 4*unit+gate per CTA
    alignas(64) unsigned char tmap_wtc[128];
    uint4 *frag2[2] = {nullptr, nullptr};  // H-LSTM: fragments of the gate output matrices W
    float *bias_out = nullptr;             // H-LSTM: [D][H][4] bias of the gate pre-activations
    int csr_max_slice_entries = 0;     // largest per-CTA slice (entries, padded)
    unsigned *csr_reg_ent[2] = {nullptr, nullptr};   // register-resident sparse kernel: [cta][warp][slots][32] entry words
    unsigned *csr_reg_rows[2] = {nullptr, nullptr};  //   and the lanes' rows [cta][warp][32]
    CsrLaneLists csr_lists[2];         // host side, until the slot count of the handle is known
    ProjTcPlan plan;                   // tensor-core projection plan for plan_M rows
    int plan_M = -1;
};

}  // namespace

struct lstm_handle {
    int L = 0, D = 1, in_dim = 0, H = 0, dtype = 0, exec_mode = 0, max_T = 0, max_B = 0;
    int device = 0, sm_count = 0, smem_optin = 0;
    int Hp8 = 0, Hs = 0;
    int ncta_dir = 0, upc = 0, threads = 0;
    bool use_tc = false;
    // register-resident recurrent kernel (bf16 dense): row tiles, column tiles per warp in registers and
    // in shared memory, warps per CTA
    bool use_mma = false;
    bool fuse_ok = false;              // short single sequences: projection fused into the register-resident kernel's prologue
    // register-resident sparse kernel (bf16, CSR execution): warps, columns per warp, row tiles, entry slots per lane
    bool use_csr_reg = false;
    bool csr_fuse_ok = false;          // register-resident sparse kernel: single short sequences project in its prologue
    bool csr_dense_proj = false;       // CSR handle whose input projection runs on the tensor cores over Wx with explicit zeros
    int csr_nw = 0, csr_kspan = 0, csr_mt = 0, csr_slots = 0;
    long long csr_conflicts = 0;       // shared-memory wavefronts per step and CTA lost to bank conflicts (worst CTA, worst matrix)
    int mma_mt = 0, mma_nkr = 0, mma_nks = 0, mma_nw = 0;
    // batched tensor-core recurrence (more than four batch rows): weight-tile rows, K blocks, planes, stamps
    bool seq_dirs = false;             // bidirectional layers run one direction after the other, each on all SMs
    bool use_tcb = false;
    bool tcb_pair = false;             // the batched recurrence splits K over clusters of two CTAs
    int tcb_RA = 0, tcb_nkb = 0, tcb_ld = 0, tcb_ldh = 0, tcb_mapN = 0;
    __nv_bfloat16 *hplanes = nullptr; unsigned *tcb_flags = nullptr;
    alignas(64) unsigned char tmap_planes[128];
    // H-LSTM cell: width of the hidden layer inside each gate (0: plain LSTM), pass-2 column tiles per warp
    int Hh = 0, hl_nkw2 = 0;
    unsigned long long *rxch = nullptr; size_t rxch_words = 0;
    std::vector<Layer> layers;
    // workspace
    float *G = nullptr; size_t G_cap = 0;
    __nv_bfloat16 *xb0 = nullptr; int ld0 = 0;
    __nv_bfloat16 *xbn[2] = {nullptr, nullptr}; int ldn = 0;
    float *ybuf[2] = {nullptr, nullptr};
    unsigned long long *xch = nullptr; size_t xch_words = 0;
    int *status_dev = nullptr;
    unsigned stamp_next = 1;           // stamps start at 1: a cleared exchange word or flag (0) never matches or exceeds a wanted stamp
    long long spin_limit = 2000000000LL;
    long long spin_limit_default = 2000000000LL;
    int withhold_cta = -1;             // failure-path self-test (lstm_selftest_timeout)
    int probe = 0;                     // step-cost measurement (lstm_probe): parts of the recurrent step left out
    cudaStream_t last_stream = nullptr;
    // host-buffer variant staging
    float *hx = nullptr, *hy = nullptr, *hh0 = nullptr, *hc0 = nullptr, *hhT = nullptr, *hcT = nullptr;
    int *status_pinned = nullptr;      // pinned host word the host-buffer call copies the device status into
    // profiling
    bool prof = false;
    std::vector<cudaEvent_t> ev;
    std::vector<int> ev_kind;
    int ev_used = 0;
    int last_launches = 0;
    // layer-wavefront kernel (unidirectional stacks, up to four sequences): CTAs per layer, units per CTA, tiling
    bool use_wave = false;
    int wave_ncta = 0, wave_upc = 0, wave_mt = 0, wave_nkr = 0, wave_nkw[kMaxWaveLayers] = {0, 0, 0, 0}, wave_nkw_max = 0;
    uint4 *wave_frag[kMaxWaveLayers] = {nullptr, nullptr, nullptr, nullptr};
    unsigned long long *wave_xch = nullptr; size_t wave_xch_words = 0;
    // row/column-pruned stacks: the forward pass runs on an inner handle over the surviving units (width Hc)
    lstm_handle *inner = nullptr;
    int Hc = 0, n_removed = 0;
    int *cmap = nullptr, *rem_idx = nullptr;
    float *rem_bias = nullptr;
    float *ch0 = nullptr, *cc0 = nullptr, *cy = nullptr, *chT = nullptr, *ccT = nullptr;
    std::string err;
};

namespace {

int fail(lstm_handle *h, int code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (h) h->err = buf; else g_create_error = buf;
    return code;
}

// A handle is bound to the device that was current in lstm_create: launching with another device current
// would run kernels there on this device's pointers.
int check_device(lstm_handle *h)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (dev != h->device)
        return fail(h, LSTM_ERR_INVALID, "the handle belongs to device %d but device %d is current; nothing launched", h->device, dev);
    return LSTM_OK;
}

// Returns a host-readable view of n bytes at p (copying from the device when p is device memory).
struct HostView {
    std::vector<unsigned char> copy;
    const void *ptr = nullptr;
};
bool host_view(const void *p, size_t bytes, HostView &v)
{
    v.ptr = p;
    if (!p || bytes == 0) return true;
    cudaPointerAttributes at;
    cudaError_t e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) { cudaGetLastError(); return true; }      // plain host memory on old drivers
    if (at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged) {
        v.copy.resize(bytes);
        if (cudaMemcpy(v.copy.data(), p, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return false;
        v.ptr = v.copy.data();
    }
    return true;
}

// One matrix in row-compressed host form: kept entries of each row in increasing column order.
struct HostCsr {
    std::vector<int> rowptr;
    std::vector<int> col;
    std::vector<float> val;
};

// Normalises either description of a [rows x cols] matrix into HostCsr (keep_zeros: with a mask, a
// kept entry whose value is 0 stays an entry; without mask or CSR, only non-zero values are kept).
int matrix_to_csr(lstm_handle *h, int rows, int cols, const float *dense, const uint8_t *mask,
                  const int32_t *rowptr, const int32_t *col, const float *val, HostCsr &out, const char *name)
{
    out.rowptr.assign(rows + 1, 0);
    if (rowptr) {
        HostView rp, cv, vv;
        if (!host_view(rowptr, sizeof(int32_t) * (rows + 1), rp)) return fail(h, LSTM_ERR_CUDA, "reading %s rowptr", name);
        const int32_t *r = (const int32_t *)rp.ptr;
        if (r[0] != 0) return fail(h, LSTM_ERR_INVALID, "%s: CSR rowptr[0] != 0", name);
        for (int i = 0; i < rows; ++i)
            if (r[i + 1] < r[i]) return fail(h, LSTM_ERR_INVALID, "%s: CSR rowptr decreases at row %d", name, i);
        const int nnz = r[rows];
        if (nnz > 0 && (!col || !val)) return fail(h, LSTM_ERR_INVALID, "%s: CSR col/val missing", name);
        if (!host_view(col, sizeof(int32_t) * nnz, cv) || !host_view(val, sizeof(float) * nnz, vv))
            return fail(h, LSTM_ERR_CUDA, "reading %s CSR arrays", name);
        const int32_t *c = (const int32_t *)cv.ptr;
        const float *v = (const float *)vv.ptr;
        for (int i = 0; i < rows; ++i)
            for (int e = r[i]; e < r[i + 1]; ++e) {
                if (c[e] < 0 || c[e] >= cols) return fail(h, LSTM_ERR_INVALID, "%s: CSR column %d out of range in row %d", name, c[e], i);
                if (e > r[i] && c[e] <= c[e - 1]) return fail(h, LSTM_ERR_INVALID, "%s: CSR columns not strictly increasing in row %d", name, i);
            }
        out.rowptr.assign(r, r + rows + 1);
        out.col.assign(c, c + nnz);
        out.val.assign(v, v + nnz);
        return LSTM_OK;
    }
    if (!dense) return fail(h, LSTM_ERR_INVALID, "%s: neither dense nor CSR weights given", name);
    HostView dv, mv;
    if (!host_view(dense, sizeof(float) * (size_t)rows * cols, dv) || !host_view(mask, (size_t)rows * cols, mv))
        return fail(h, LSTM_ERR_CUDA, "reading %s", name);
    const float *w = (const float *)dv.ptr;
    const uint8_t *m = (const uint8_t *)mv.ptr;
    for (int i = 0; i < rows; ++i) {
        for (int k = 0; k < cols; ++k) {
            const size_t idx = (size_t)i * cols + k;
            const bool keep = m ? (m[idx] != 0) : (w[idx] != 0.0f);
            if (keep) { out.col.push_back(k); out.val.push_back(w[idx]); }
        }
        out.rowptr[i + 1] = (int)out.col.size();
    }
    return LSTM_OK;
}

// Dense [rows x cols] fp32 with the mask applied as explicit zeros (W (x) Msk), from either form.
int matrix_to_dense(lstm_handle *h, int rows, int cols, const float *dense, const uint8_t *mask,
                    const int32_t *rowptr, const int32_t *col, const float *val, std::vector<float> &out,
                    const char *name)
{
    out.assign((size_t)rows * cols, 0.0f);
    if (rowptr) {
        HostCsr c;
        int rc = matrix_to_csr(h, rows, cols, nullptr, nullptr, rowptr, col, val, c, name);
        if (rc) return rc;
        for (int i = 0; i < rows; ++i)
            for (int e = c.rowptr[i]; e < c.rowptr[i + 1]; ++e) out[(size_t)i * cols + c.col[e]] = c.val[e];
        return LSTM_OK;
    }
    if (!dense) return fail(h, LSTM_ERR_INVALID, "%s: neither dense nor CSR weights given", name);
    HostView dv, mv;
    if (!host_view(dense, sizeof(float) * (size_t)rows * cols, dv) || !host_view(mask, (size_t)rows * cols, mv))
        return fail(h, LSTM_ERR_CUDA, "reading %s", name);
    const float *w = (const float *)dv.ptr;
    const uint8_t *m = (const uint8_t *)mv.ptr;
    for (size_t i = 0; i < out.size(); ++i) out[i] = (m && !m[i]) ? 0.0f : w[i];
    return LSTM_OK;
}

template <typename T>
int upload(lstm_handle *h, T **dst, const void *src, size_t bytes, cudaStream_t st, const char *what)
{
    *dst = nullptr;
    if (cudaMalloc((void **)dst, bytes ? bytes : 16) != cudaSuccess) {
        cudaGetLastError();
        return fail(h, LSTM_ERR_NOMEM, "device allocation of %zu bytes for %s failed", bytes, what);
    }
    if (bytes && cudaMemcpyAsync(*dst, src, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return fail(h, LSTM_ERR_CUDA, "upload of %s failed: %s", what, cudaGetErrorString(cudaGetLastError()));
    // the source vectors are pageable host memory: the async copy stages them before returning
    return LSTM_OK;
}

template <typename T>
int dev_alloc(lstm_handle *h, T **dst, size_t bytes, bool zero, cudaStream_t st, const char *what)
{
    *dst = nullptr;
    if (cudaMalloc((void **)dst, bytes ? bytes : 16) != cudaSuccess) {
        cudaGetLastError();
        return fail(h, LSTM_ERR_NOMEM, "device allocation of %zu bytes for %s failed", bytes, what);
    }
    if (zero && bytes && cudaMemsetAsync(*dst, 0, bytes, st) != cudaSuccess)
        return fail(h, LSTM_ERR_CUDA, "clearing %s failed", what);
    return LSTM_OK;
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

void unit_range_host(int H, int nc, int c, int &u0, int &n)
{
    const int base = H / nc, rem = H % nc;
    n = base + (c < rem ? 1 : 0);
    u0 = c * base + std::min(c, rem);
}

// Launch shape of the recurrent kernel for B batch rows.
struct RecurShape { int BT; size_t smem; int w_smem_bytes; int units_res_min; bool staged = false; bool stage_all = false; int threads = 0; };

RecurShape recur_shape(const lstm_handle *h, int B, int layer)
{
    if (h->use_mma) {
        RecurShape s;
        s.BT = 4;
        // several batch rows: the exchange words land in shared memory (16-byte copies need an even H,
        // at most 12 pairs per lane, and room for the landing area)
        const int kspan = (h->mma_nkr + h->mma_nks) * 16;
        s.staged = B > 1 && (h->H % 2) == 0 && 4 * kspan <= 64 * 12 &&
                   recur_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->upc, B, true) <= (size_t)h->smem_optin - 64;
        s.smem = recur_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->upc, B, s.staged);
        s.w_smem_bytes = h->mma_nw * h->mma_nks * h->mma_mt * 512;
        s.units_res_min = 0;
        return s;
    }
    const size_t budget = (size_t)h->smem_optin - 64;            // static shared memory of the kernel
    const bool csr = h->exec_mode == LSTM_CSR;
    const size_t wsize = h->dtype == LSTM_BF16W_F32S ? 2 : 4;
    size_t need_w;
    if (!csr) need_w = (size_t)h->upc * 4 * h->Hp8 * wsize;
    else {
        const size_t esize = h->dtype == LSTM_BF16W_F32S ? 4 : 8;
        need_w = (size_t)round_up(4 * h->upc + 1, 4) * 4 + (size_t)h->layers[layer].csr_max_slice_entries * esize;
    }
    const size_t c_bytes = (size_t)round_up(h->upc * B, 4) * 4;
    auto fixed = [&](int bt) { return (size_t)2 * bt * h->Hs * 4 + c_bytes; };
    // candidates in order of preference: cost per weight ~ chunks * (1 unpack + BT FMAs)
    int cands[4]; int nc = 0;
    if (B <= 1) cands[nc++] = 1;
    else if (B == 2) { cands[nc++] = 2; cands[nc++] = 1; }
    else if (B <= 4) { cands[nc++] = 4; cands[nc++] = 2; cands[nc++] = 1; }
    else if (h->dtype == LSTM_F32) { cands[nc++] = 4; cands[nc++] = 2; cands[nc++] = 1; }   // fp64 accumulators
    else {
        const int c8 = ((B + 7) / 8) * 9, c4 = ((B + 3) / 4) * 5;
        if (c8 <= c4) { cands[nc++] = 8; cands[nc++] = 4; } else { cands[nc++] = 4; cands[nc++] = 8; }
        cands[nc++] = 2; cands[nc++] = 1;
    }
    int pick = cands[nc - 1];
    for (int i = 0; i < nc; ++i)
        if (fixed(cands[i]) + need_w <= budget) { pick = cands[i]; break; }
    RecurShape s;
    s.BT = pick;
    const size_t f = fixed(pick);
    const size_t avail = budget > f ? budget - f : 0;
    const size_t w = std::min(need_w, avail);
    s.w_smem_bytes = (int)w;
    s.smem = f + w;
    s.units_res_min = 0;
    s.threads = h->threads;
    // several chunks of rows per step: when all B rows of h fit beside the whole slice, they are staged at once
    // (one polling phase per step instead of one per chunk) and the (unit, chunk) pairs spread over the warps
    const size_t f_all = (size_t)2 * round_up(B, pick) * h->Hs * 4 + c_bytes;      // whole chunks of rows per buffer
    if (B > pick && f_all + need_w <= budget) {
        s.stage_all = true;
        s.smem = f_all + need_w;
        s.w_smem_bytes = (int)need_w;
        const int nchunk = (B + pick - 1) / pick;
        (void)nchunk;
        s.threads = 512;                 // all hands for the one polling phase: B * H words, eight per thread in flight
    }
    return s;
}

// Chooses the tiling of the register-resident recurrent kernel, or leaves use_mma false when the
// slice of a CTA does not fit registers + shared memory (then the shared-memory kernel runs).
void plan_mma(lstm_handle *h)
{
    h->use_mma = false;
    if (h->dtype != LSTM_BF16W_F32S || h->exec_mode != LSTM_DENSE) return;
    const char *env = getenv("LSTM_B200_RECUR");
    if (env && strcmp(env, "simt") == 0) return;      // LSTM_B200_RECUR=simt selects the shared-memory kernel
    const int mt = (4 * h->upc + 15) / 16;
    if (mt > 4) return;
    const int nk = (h->H + 15) / 16;
    const int nw = (nk <= 32 && h->upc <= 8) ? 8 : 16;   // warp w also finishes unit w: upc <= warps
    if (h->upc > nw) return;
    const int need = (nk + nw - 1) / nw;               // column tiles per warp
    const int cap = (nw == 16 ? kMmaTileCap16 : kMmaTileCap8) / mt;
    int nkr = 0;
    for (int c = 2; c <= 8; c += 2)
        if (c <= cap && (nkr == 0 || nkr < need)) nkr = c;     // smallest even count >= need, else the largest allowed
    if (nkr == 0) return;
    const int nks = need > nkr ? need - nkr : 0;
    if (!recur_mma_shape_ok(mt, nkr, nw)) return;
    if (recur_mma_smem_bytes(mt, nkr, nw, nks, h->upc, h->max_B, false) > (size_t)h->smem_optin - 64) return;
    h->use_mma = true;
    h->mma_mt = mt; h->mma_nkr = nkr; h->mma_nks = nks; h->mma_nw = nw;
}

int max_b_fits(const lstm_handle *h)
{
    if (h->use_mma || h->use_csr_reg) return 1;
    // the staging buffers and the c state must fit even when no weight is resident
    const size_t budget = (size_t)h->smem_optin - 64;
    const size_t c_bytes = (size_t)round_up(h->upc * h->max_B, 4) * 4;
    const size_t rp = h->exec_mode == LSTM_CSR ? (size_t)round_up(4 * h->upc + 1, 4) * 4 : 0;
    return (size_t)2 * h->Hs * 4 + c_bytes + rp <= budget;
}

// Operand-A fragments of a [4U x K] matrix whose row q*U + u is gate q of unit u: per CTA (units split
// evenly over ncta CTAs) [warp][column tile][row tile][lane] x 4 words, local row = 4 * unit + gate,
// zero beyond the CTA's units and beyond column K.
std::vector<uint32_t> pack_fragments(const float *m, int U, int K, int ncta, int NW, int nkw, int MT, bool adjacent = false)
{
    std::vector<uint32_t> f((size_t)ncta * NW * nkw * MT * 32 * 4, 0u);
    size_t o = 0;
    for (int c = 0; c < ncta; ++c) {
        int u0, nu; unit_range_host(U, ncta, c, u0, nu);
        auto wv = [&](int r, int k) -> uint32_t {
            if (r >= 4 * nu || k >= K) return 0u;
            return f32_to_bf16_rne(m[(size_t)((r & 3) * U + u0 + (r >> 2)) * K + k]);
        };
        for (int wp = 0; wp < NW; ++wp)
            for (int i = 0; i < nkw; ++i)
                for (int mt = 0; mt < MT; ++mt)
                    for (int lane = 0; lane < 32; ++lane) {
                        const int g = lane >> 2, p2 = (lane & 3) * 2;
                        const int r0 = mt * 16 + g, r1 = r0 + 8;
                        // adjacent: the lane's four MMA k slots hold the adjacent columns 4 * (lane & 3) .. + 3 (the
                        // input-projection fragments, whose other operand is then one 16-byte load)
                        const int ka = (wp * nkw + i) * 16 + (adjacent ? 2 * p2 : p2), kb = adjacent ? ka + 2 : ka + 8;
                        f[o++] = wv(r0, ka) | (wv(r0, ka + 1) << 16);
                        f[o++] = wv(r1, ka) | (wv(r1, ka + 1) << 16);
                        f[o++] = wv(r0, kb) | (wv(r0, kb + 1) << 16);
                        f[o++] = wv(r1, kb) | (wv(r1, kb + 1) << 16);
                    }
    }
    return f;
}

// Tiling of the layer-wavefront kernel, or use_wave = false when the stack does not qualify: one direction, two
// to four layers, bf16 dense, at most 16 units per CTA with the SMs split evenly between the layers, and the
// widest layer's slice (4 * units rows by 2H columns) inside registers + shared memory.
void plan_wave(lstm_handle *h)
{
    h->use_wave = false;
    if (h->D != 1 || h->L < 2 || h->L > kMaxWaveLayers || h->dtype != LSTM_BF16W_F32S || h->exec_mode != LSTM_DENSE || h->Hh) return;
    const char *env = getenv("LSTM_B200_WAVE");
    if (env && strcmp(env, "0") == 0) return;
    const int H = h->H;
    const int n = std::max(1, std::min(h->sm_count / h->L, H));
    const int upc = (H + n - 1) / n;
    if (upc > 16) return;
    const int mt = (4 * upc + 15) / 16;
    const int need0 = ((H + 15) / 16 + 15) / 16, need1 = ((2 * H + 15) / 16 + 15) / 16;
    const int cap = kWaveTileCap / mt;
    int nkr = 0;
    for (int c = 2; c <= 8; c += 2)
        if (c <= cap && (nkr == 0 || nkr < need1)) nkr = c;
    if (nkr == 0 || !recur_wave_shape_ok(mt, nkr)) return;
    const int nkw0 = std::max(need0, nkr), nkw1 = std::max(need1, nkr);
    if (recur_wave_smem_bytes(mt, nkr, nkw1, upc, std::min(h->max_B, 4)) > (size_t)h->smem_optin - 64) return;
    h->use_wave = true;
    h->wave_ncta = n; h->wave_upc = upc; h->wave_mt = mt; h->wave_nkr = nkr; h->wave_nkw_max = nkw1;
    for (int l = 0; l < h->L; ++l) h->wave_nkw[l] = l == 0 ? nkw0 : nkw1;
}

void free_all(lstm_handle *h)
{
    for (auto &ly : h->layers) {
        cudaFree(ly.wx); cudaFree(ly.bias); cudaFree(ly.wx_rowptr); cudaFree(ly.wx_ent);
        for (int d = 0; d < 2; ++d) { cudaFree(ly.wh[d]); cudaFree(ly.wh_ptr[d]); cudaFree(ly.wh_ent[d]); cudaFree(ly.wfrag[d]); cudaFree(ly.xfrag[d]); cudaFree(ly.frag2[d]); cudaFree(ly.csr_reg_ent[d]); cudaFree(ly.csr_reg_rows[d]); }
        cudaFree(ly.bias_out); cudaFree(ly.wtc);
    }
    cudaFree(h->G); cudaFree(h->xb0); cudaFree(h->xbn[0]); cudaFree(h->xbn[1]);
    cudaFree(h->ybuf[0]); cudaFree(h->ybuf[1]); cudaFree(h->xch); cudaFree(h->rxch); cudaFree(h->hplanes); cudaFree(h->tcb_flags); cudaFree(h->status_dev);
    for (int l = 0; l < kMaxWaveLayers; ++l) cudaFree(h->wave_frag[l]);
    cudaFree(h->wave_xch);
    cudaFree(h->cmap); cudaFree(h->rem_idx); cudaFree(h->rem_bias);
    cudaFree(h->ch0); cudaFree(h->cc0); cudaFree(h->cy); cudaFree(h->chT); cudaFree(h->ccT);
    if (h->status_pinned) cudaFreeHost(h->status_pinned);
    cudaFree(h->hx); cudaFree(h->hy); cudaFree(h->hh0); cudaFree(h->hc0); cudaFree(h->hhT); cudaFree(h->hcT);
    for (auto e : h->ev) cudaEventDestroy(e);
    cudaGetLastError();
}

bool want_tc(const lstm_handle *h)
{
    if (h->dtype != LSTM_BF16W_F32S || h->exec_mode != LSTM_DENSE) return false;
    const char *env = getenv("LSTM_B200_PROJ");
    return !(env && strcmp(env, "simt") == 0);     // LSTM_B200_PROJ=simt selects the CUDA-core projection
}

int n_split_cap() { return 4; }

}  // namespace

extern "C" {

const char *lstm_last_error(const lstm_handle *h) { return h ? h->err.c_str() : g_create_error.c_str(); }

static int try_compaction(lstm_handle **out, int layers, int in_dim, int hidden, int bidir, int dtype,
                          const lstm_weights *w, int exec_mode, int max_T, int max_B, void *cuda_stream, bool *done);

static int create_impl(lstm_handle **out, int layers, int in_dim, int hidden, int bidir, int dtype,
                       const lstm_weights *w, int exec_mode, int max_T, int max_B, void *cuda_stream, bool allow_compact)
{
    if (!out) return fail(nullptr, LSTM_ERR_INVALID, "out is NULL");
    *out = nullptr;
    if (layers < 1 || in_dim < 1 || hidden < 1 || (bidir != 0 && bidir != 1) || !w || max_T < 1 || max_B < 1)
        return fail(nullptr, LSTM_ERR_INVALID, "bad argument: layers=%d in_dim=%d hidden=%d bidir=%d max_T=%d max_B=%d w=%p",
                    layers, in_dim, hidden, bidir, max_T, max_B, (const void *)w);
    if (dtype != LSTM_F32 && dtype != LSTM_BF16W_F32S) return fail(nullptr, LSTM_ERR_INVALID, "unknown dtype %d", dtype);
    if (exec_mode != LSTM_DENSE && exec_mode != LSTM_CSR) return fail(nullptr, LSTM_ERR_INVALID, "unknown exec_mode %d", exec_mode);
    if (hidden >= 65536) return fail(nullptr, LSTM_ERR_UNSUPPORTED, "hidden must be < 65536");
    if ((long long)max_T * max_B > (1LL << 30)) return fail(nullptr, LSTM_ERR_UNSUPPORTED, "max_T*max_B too large");

    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        const char *m = cudaGetErrorString(cudaGetLastError());
        return fail(nullptr, LSTM_ERR_CUDA, "no usable CUDA device: %s", m);
    }
    if (prop.major != 10) return fail(nullptr, LSTM_ERR_CUDA, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
    int coop = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (!coop) return fail(nullptr, LSTM_ERR_CUDA, "device does not support cooperative launch");

    if (allow_compact) {
        // row/column-pruned weights: run on the surviving units only (LSTM_B200_COMPACT=0 keeps the zeros)
        // Unset: only handles made for batches (max_B of five or more), where the step is bound by throughput and a
        // narrower model is faster; for up to four sequences the step is bound by the exchange latency, the narrower
        // model gains nothing and the extra scatter kernel costs a few microseconds (measured: 172.7 against 164.6 us
        // per sequence at width 1500 -> 1197).  LSTM_B200_COMPACT=1 compacts always, =0 never.
        const char *env = getenv("LSTM_B200_COMPACT");
        const bool want = env ? strcmp(env, "0") != 0 : max_B >= 5;
        if (want) {
            bool done = false;
            const int crc = try_compaction(out, layers, in_dim, hidden, bidir, dtype, w, exec_mode, max_T, max_B, cuda_stream, &done);
            if (crc != LSTM_OK || done) return crc;
        }
    }

    lstm_handle *h = new (std::nothrow) lstm_handle;
    if (!h) return fail(nullptr, LSTM_ERR_NOMEM, "host allocation failed");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->L = layers; h->D = bidir ? 2 : 1; h->in_dim = in_dim; h->H = hidden; h->dtype = dtype;
    h->exec_mode = exec_mode; h->max_T = max_T; h->max_B = max_B; h->device = dev;
    h->sm_count = prop.multiProcessorCount;
    h->smem_optin = (int)prop.sharedMemPerBlockOptin;
    h->last_stream = st;
    const int H = hidden, D = h->D;
    const bool bf16 = dtype == LSTM_BF16W_F32S;
    const bool csr = exec_mode == LSTM_CSR;
    h->Hp8 = round_up(H, 8);
    h->Hs = round_up(H, 256);
    h->ncta_dir = std::max(1, std::min(h->sm_count / D, H));
    if (const char *e = getenv("LSTM_B200_CTAS")) {     // measurement: fewer CTAs per direction than SMs
        const int want = atoi(e);
        if (want >= 1 && want <= h->ncta_dir) h->ncta_dir = want;
    }
    h->upc = (H + h->ncta_dir - 1) / h->ncta_dir;
    // fp32 storage: no more CTAs than full slices (H = 200: 100 CTAs of two units, not 52 of two and 96 of one).
    // The step waits for the slowest CTA either way, and every CTA less is B * H fewer words polled per step
    // (workload 1: 6.8 -> 5.3 us per step).
    if (dtype == LSTM_F32) h->ncta_dir = (H + h->upc - 1) / h->upc;
    h->threads = std::max(128, 32 * std::min(h->upc, 16));
    h->use_tc = want_tc(h);
    {
        // A pruned Wx still makes a dense contraction with all timesteps as the other operand, and at the densities
        // pruning reaches (0.05 .. 0.10) the tensor cores multiply the zeros faster than CUDA cores walk the lists
        // (the paper's own observation about sparse matmuls on GPUs, Section 3): bf16 CSR handles keep a dense
        // copy of Wx for the projection; the recurrence, where the lists stay on-chip, remains sparse.
        // LSTM_B200_PROJ=csr keeps the list-walking projection, =simt the CUDA-core dense one.
        const char *env = getenv("LSTM_B200_PROJ");
        h->csr_dense_proj = csr && bf16 && !(env && (strcmp(env, "csr") == 0 || strcmp(env, "simt") == 0));
        if (h->csr_dense_proj) h->use_tc = true;
    }
    plan_mma(h);
    plan_wave(h);
    {
        const char *env = getenv("LSTM_B200_FUSE");
        h->fuse_ok = h->use_mma && !(env && strcmp(env, "0") == 0) &&
                     recur_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->upc, 1, false, true) <= (size_t)h->smem_optin - 64;
    }
    if (csr && bf16) {
        // the register-resident sparse kernel: at most 16 units per CTA (warp w finishes unit w, a lane owns at
        // most two of the 4 * units rows); the entry slots per lane are known once every matrix has been laid out
        const char *env = getenv("LSTM_B200_RECUR");
        const int nw = (h->upc <= 8 && H <= 512) ? 8 : 16;
        const int kspan = round_up((H + nw - 1) / nw, 32), mt = (4 * h->upc + 15) / 16;
        if (!(env && strcmp(env, "simt") == 0) && h->upc <= nw &&
            recur_csr_reg_smem_bytes(nw, kspan, mt, h->upc, max_B) <= (size_t)h->smem_optin - 64) {
            h->use_csr_reg = true; h->csr_nw = nw; h->csr_kspan = kspan; h->csr_mt = mt;
            const char *fenv = getenv("LSTM_B200_FUSE");
            h->csr_fuse_ok = h->csr_dense_proj && nw == 16 && mt <= 4 && !(fenv && strcmp(fenv, "0") == 0) &&
                             recur_csr_reg_fuse_smem_bytes(nw, kspan, mt, h->upc) <= (size_t)h->smem_optin - 64;
        }
    }
    // does the batched tensor-core recurrence fit with the current split of the SMs?
    auto tcb_fits = [&](int *kbs, int *stages) -> bool {
        const char *env = getenv("LSTM_B200_RECUR");
        const int RA = round_up(4 * h->upc, 8), nkb = (H + 63) / 64;
        if (!(bf16 && !csr && max_B > 4 && RA <= 128) || (env && (strcmp(env, "mma") == 0 || strcmp(env, "simt") == 0))) return false;
        const int B = std::min(max_B, 32), N = round_up(2 * B, 16);
        return h->ncta_dir <= 160 && recur_tc_plan(RA, nkb, N, h->upc, B, (size_t)h->smem_optin - kTcStaticSmem, 0, kbs, stages);
    };
    int kbs_tmp = 0, stages_tmp = 0;
    if (D == 2 && bf16 && !csr && !h->use_mma && !tcb_fits(&kbs_tmp, &stages_tmp)) {
        // Side by side, each direction has half the SMs and a slice twice as tall; when that slice fits
        // neither the register-resident kernel nor (for handles made for batches) the tensor-core one, run
        // the directions one after the other on all SMs instead: twice the steps, but every step on-chip.
        const int nc = h->ncta_dir, up = h->upc, th = h->threads;
        h->ncta_dir = std::max(1, std::min(h->sm_count, H));
        h->upc = (H + h->ncta_dir - 1) / h->ncta_dir;
        h->threads = std::max(128, 32 * std::min(h->upc, 16));
        plan_mma(h);
        if (h->use_mma) h->seq_dirs = true;
        else { h->ncta_dir = nc; h->upc = up; h->threads = th; }
    }
    if (tcb_fits(&kbs_tmp, &stages_tmp)) {   // batched tensor-core recurrence, beside the kernels for up to four sequences
        h->use_tcb = true; h->tcb_RA = round_up(4 * h->upc, 8); h->tcb_nkb = (H + 63) / 64; h->tcb_ld = h->tcb_nkb * 64;
        h->tcb_ldh = round_up(H, 64);      // rows of the planes start on 128-byte lines: a TMA box row is one line, not two
        // pair mode: two CTAs of a cluster split K (half the tensor instructions per step) when the pairs do
        // not straddle directions, the doubled tile fits, and the device can co-schedule the clusters
        const char *env = getenv("LSTM_B200_RECUR");
        const int Bp = std::min(max_B, 32), Np = round_up(2 * Bp, 16);
        int kp = 0, sp = 0;
        // a pair's tile holds both CTAs' rows back to back: 2 x 4 x units is already a multiple of the 8-row swizzle
        // group, so the rows are not padded (at 11 units per CTA the 8 rows saved per K block let the ring hold a
        // whole step's operand)
        const int RAp = 4 * h->upc;
        if (!(env && strcmp(env, "tc1") == 0) && (h->ncta_dir % 2) == 0 &&
            recur_tc_plan(RAp, h->tcb_nkb, Np, h->upc, Bp, (size_t)h->smem_optin - kTcStaticSmem, 1, &kp, &sp) &&
            recur_tc_prepare(h->smem_optin - kTcStaticSmem) == cudaSuccess &&
            recur_tc_pair_supported(h->ncta_dir * (h->seq_dirs ? 1 : D), recur_tc_smem_bytes(RAp, h->tcb_nkb, Np, sp, kp, h->upc, Bp, 1))) {
            h->tcb_pair = true;
            h->tcb_RA = RAp;
        }
    }
    h->layers.resize(layers);
    if (const char *env = getenv("LSTM_B200_SPIN_LIMIT")) { long long v = atoll(env); if (v > 0) h->spin_limit = v; }
    h->spin_limit_default = h->spin_limit;

    int rc = LSTM_OK;
    auto bail = [&](int code) { g_create_error = h->err; free_all(h); delete h; return code; };
    if (!max_b_fits(h)) { fail(h, LSTM_ERR_UNSUPPORTED, "hidden=%d with max_B=%d does not fit the recurrent kernel's shared memory", H, max_B); return bail(LSTM_ERR_UNSUPPORTED); }

    for (int l = 0; l < layers && rc == LSTM_OK; ++l) {
        Layer &ly = h->layers[l];
        ly.in_l = l == 0 ? in_dim : D * H;
        ly.ldk = bf16 ? round_up(ly.in_l, 8) : ly.in_l;
        if (csr && (size_t)ly.in_l * 8 * 4 > (size_t)h->smem_optin) { rc = fail(h, LSTM_ERR_UNSUPPORTED, "sparse projection supports input widths up to %d", h->smem_optin / 32); break; }
        const int N = D * 4 * H;
        std::vector<float> bias_p((size_t)N, 0.0f);
        std::vector<uint16_t> wx16; std::vector<float> wx32;
        std::vector<int> px_rowptr; std::vector<CsrEntry> px_ent;
        std::vector<uint16_t> tcb_rows;
        if (!csr) { if (bf16) wx16.assign((size_t)N * ly.ldk, 0); else wx32.assign((size_t)N * ly.ldk, 0.0f); }
        else { px_rowptr.assign(N + 1, 0); if (h->csr_dense_proj) wx16.assign((size_t)N * ly.ldk, 0); }

        for (int d = 0; d < D && rc == LSTM_OK; ++d) {
            const lstm_weights &src = w[l * D + d];
            char name[64];
            // bias
            if (src.b) {
                HostView bv;
                if (!host_view(src.b, sizeof(float) * 4 * H, bv)) { rc = fail(h, LSTM_ERR_CUDA, "reading bias"); break; }
                const float *b = (const float *)bv.ptr;
                for (int q = 0; q < 4; ++q)
                    for (int j = 0; j < H; ++j) bias_p[(size_t)d * 4 * H + (size_t)j * 4 + q] = b[q * H + j];
            }
            if (!csr) {
                std::vector<float> m;
                snprintf(name, sizeof name, "wx[layer %d, dir %d]", l, d);
                rc = matrix_to_dense(h, 4 * H, ly.in_l, src.wx, src.mask_x, src.wx_rowptr, src.wx_col, src.wx_val, m, name);
                if (rc) break;
                std::vector<float> wave_x;
                if (h->use_wave && l > 0) wave_x = m;                 // the wavefront kernel folds Wx of the upper layers into the step
                if (h->use_mma && bf16 && h->fuse_ok) {
                    // the same matrix as operand-A fragments: short single sequences compute their projection in the
                    // recurrent kernel's prologue
                    const int nranges = h->mma_nw / 2;                 // two warps share a column range
                    ly.nkw_x = ((ly.in_l + 15) / 16 + nranges - 1) / nranges;
                    const std::vector<uint32_t> fx = pack_fragments(m.data(), H, ly.in_l, h->ncta_dir, nranges, ly.nkw_x, h->mma_mt, true);
                    rc = upload(h, (uint32_t **)&ly.xfrag[d], fx.data(), fx.size() * 4, st, "input weight fragments");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                    if (rc) break;
                }
                for (int q = 0; q < 4; ++q)
                    for (int j = 0; j < H; ++j) {
                        const float *srow = m.data() + (size_t)(q * H + j) * ly.in_l;
                        const size_t drow = ((size_t)d * 4 * H + (size_t)j * 4 + q) * ly.ldk;
                        if (bf16) for (int k = 0; k < ly.in_l; ++k) wx16[drow + k] = f32_to_bf16_rne(srow[k]);
                        else memcpy(&wx32[drow], srow, sizeof(float) * ly.in_l);
                    }
                snprintf(name, sizeof name, "wh[layer %d, dir %d]", l, d);
                rc = matrix_to_dense(h, 4 * H, H, src.wh, src.mask_h, src.wh_rowptr, src.wh_col, src.wh_val, m, name);
                if (rc) break;
                if (h->use_wave) {
                    // layer 0: Wh alone; above: [Wx | Wh] side by side, 2H columns
                    std::vector<float> cat;
                    const float *src_m = m.data();
                    int Kw = H;
                    if (l > 0) {
                        Kw = 2 * H;
                        cat.resize((size_t)4 * H * Kw);
                        for (int r = 0; r < 4 * H; ++r) {
                            memcpy(cat.data() + (size_t)r * Kw, wave_x.data() + (size_t)r * H, sizeof(float) * H);
                            memcpy(cat.data() + (size_t)r * Kw + H, m.data() + (size_t)r * H, sizeof(float) * H);
                        }
                        src_m = cat.data();
                    }
                    const std::vector<uint32_t> f = pack_fragments(src_m, H, Kw, h->wave_ncta, 16, h->wave_nkw[l], h->wave_mt);
                    rc = upload(h, (uint32_t **)&h->wave_frag[l], f.data(), f.size() * 4, st, "wavefront weight fragments");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                    if (rc) break;
                }
                const size_t n = (size_t)H * 4 * h->Hp8;
                if (h->use_mma) {
                    const std::vector<uint32_t> f = pack_fragments(m.data(), H, H, h->ncta_dir, h->mma_nw, h->mma_nkr + h->mma_nks, h->mma_mt);
                    rc = upload(h, (uint32_t **)&ly.wfrag[d], f.data(), f.size() * 4, st, "recurrent weight fragments");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                } else if (bf16) {
                    std::vector<uint16_t> p(n, 0);
                    for (int j = 0; j < H; ++j)
                        for (int q = 0; q < 4; ++q) {
                            const float *srow = m.data() + (size_t)(q * H + j) * H;
                            uint16_t *drow = p.data() + ((size_t)j * 4 + q) * h->Hp8;
                            for (int k = 0; k < H; ++k) drow[k] = f32_to_bf16_rne(srow[k]);
                        }
                    rc = upload(h, &ly.wh[d], p.data(), n * 2, st, "recurrent weights");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                } else {
                    std::vector<float> p(n, 0.0f);
                    for (int j = 0; j < H; ++j)
                        for (int q = 0; q < 4; ++q)
                            memcpy(p.data() + ((size_t)j * 4 + q) * h->Hp8, m.data() + (size_t)(q * H + j) * H, sizeof(float) * H);
                    rc = upload(h, &ly.wh[d], p.data(), n * 4, st, "recurrent weights");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                }
                if (rc == LSTM_OK && h->use_tcb) {
                    // the same slices as plain K-major rows for the tensor-core kernel's TMA tiles
                    const size_t rows_dir = (size_t)h->ncta_dir * h->tcb_RA;
                    if (d == 0) tcb_rows.assign((size_t)D * rows_dir * h->tcb_ld, 0);
                    for (int c = 0; c < h->ncta_dir; ++c) {
                        int u0, nu; unit_range_host(H, h->ncta_dir, c, u0, nu);
                        for (int u = 0; u < nu; ++u)
                            for (int q = 0; q < 4; ++q) {
                                const float *srow = m.data() + (size_t)(q * H + u0 + u) * H;
                                uint16_t *drow = tcb_rows.data() + ((size_t)d * rows_dir + (size_t)c * h->tcb_RA + 4 * u + q) * h->tcb_ld;
                                for (int k = 0; k < H; ++k) drow[k] = f32_to_bf16_rne(srow[k]);
                            }
                    }
                }
            } else {
                HostCsr cx, ch;
                snprintf(name, sizeof name, "wx[layer %d, dir %d]", l, d);
                rc = matrix_to_csr(h, 4 * H, ly.in_l, src.wx, src.mask_x, src.wx_rowptr, src.wx_col, src.wx_val, cx, name);
                if (rc) break;
                for (int j = 0; j < H; ++j)
                    for (int q = 0; q < 4; ++q) {
                        const int r = q * H + j;
                        for (int e = cx.rowptr[r]; e < cx.rowptr[r + 1]; ++e) {
                            float v = cx.val[e];
                            if (bf16) v = bf16_to_f32(f32_to_bf16_rne(v));
                            px_ent.push_back(CsrEntry{v, cx.col[e]});
                            if (h->csr_dense_proj) wx16[((size_t)d * 4 * H + (size_t)j * 4 + q) * ly.ldk + cx.col[e]] = f32_to_bf16_rne(cx.val[e]);
                        }
                        px_rowptr[(size_t)d * 4 * H + (size_t)j * 4 + q + 1] = (int)px_ent.size();
                    }
                if (h->csr_fuse_ok) {
                    // Wx with its zeros as operand-A fragments: single short sequences project in the sparse
                    // recurrent kernel's prologue, on the tensor cores (two warps share a column range)
                    std::vector<float> m((size_t)4 * H * ly.in_l, 0.0f);
                    for (int r = 0; r < 4 * H; ++r)
                        for (int e = cx.rowptr[r]; e < cx.rowptr[r + 1]; ++e) m[(size_t)r * ly.in_l + cx.col[e]] = cx.val[e];
                    const int nranges = h->csr_nw / 2;
                    ly.nkw_x = ((ly.in_l + 15) / 16 + nranges - 1) / nranges;
                    const std::vector<uint32_t> fx = pack_fragments(m.data(), H, ly.in_l, h->ncta_dir, nranges, ly.nkw_x, h->csr_mt, true);
                    rc = upload(h, (uint32_t **)&ly.xfrag[d], fx.data(), fx.size() * 4, st, "input weight fragments");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                    if (rc) break;
                }
                snprintf(name, sizeof name, "wh[layer %d, dir %d]", l, d);
                rc = matrix_to_csr(h, 4 * H, H, src.wh, src.mask_h, src.wh_rowptr, src.wh_col, src.wh_val, ch, name);
                if (rc) break;
                if (h->use_csr_reg) {
                    csr_lane_lists(ch.rowptr.data(), ch.col.data(), ch.val.data(), H, h->ncta_dir, h->csr_nw, h->csr_kspan, ly.csr_lists[d]);
                    h->csr_slots = std::max(h->csr_slots, ly.csr_lists[d].longest);
                }
                std::vector<int> ptr(4 * H + 1, 0);
                std::vector<unsigned> e16; std::vector<CsrEntry> e32;
                for (int j = 0; j < H; ++j)
                    for (int q = 0; q < 4; ++q) {
                        const int r = q * H + j;
                        int cnt = 0;
                        for (int e = ch.rowptr[r]; e < ch.rowptr[r + 1]; ++e, ++cnt) {
                            if (bf16) e16.push_back(((unsigned)ch.col[e] << 16) | f32_to_bf16_rne(ch.val[e]));
                            else e32.push_back(CsrEntry{ch.val[e], ch.col[e]});
                        }
                        for (; cnt % 4; ++cnt) { if (bf16) e16.push_back(0u); else e32.push_back(CsrEntry{0.0f, 0}); }
                        ptr[(size_t)j * 4 + q + 1] = (int)(bf16 ? e16.size() : e32.size());
                    }
                for (int c = 0; c < h->ncta_dir; ++c) {
                    int u0, n; unit_range_host(H, h->ncta_dir, c, u0, n);
                    ly.csr_max_slice_entries = std::max(ly.csr_max_slice_entries, ptr[4 * (u0 + n)] - ptr[4 * u0]);
                }
                rc = upload(h, &ly.wh_ptr[d], ptr.data(), ptr.size() * sizeof(int), st, "recurrent CSR offsets");
                if (rc == LSTM_OK) {
                    if (bf16) rc = upload(h, (unsigned **)&ly.wh_ent[d], e16.data(), e16.size() * 4, st, "recurrent CSR entries");
                    else rc = upload(h, (CsrEntry **)&ly.wh_ent[d], e32.data(), e32.size() * 8, st, "recurrent CSR entries");
                }
                if (rc == LSTM_OK) cudaStreamSynchronize(st);
            }
        }
        if (rc) break;
        rc = upload(h, &ly.bias, bias_p.data(), bias_p.size() * 4, st, "bias");
        if (rc == LSTM_OK && h->use_tcb && !tcb_rows.empty()) {
            rc = upload(h, (uint16_t **)&ly.wtc, tcb_rows.data(), tcb_rows.size() * 2, st, "recurrent weight tiles");
            if (rc == LSTM_OK && !recur_tc_encode_weights(ly.tmap_wtc, ly.wtc, (long long)D * h->ncta_dir * h->tcb_RA, h->tcb_ld, h->tcb_pair ? 2 * h->tcb_RA : h->tcb_RA))
                rc = fail(h, LSTM_ERR_CUDA, "tensor map of the recurrent weight tiles could not be encoded");
        }
        if (rc == LSTM_OK && !csr)
            rc = bf16 ? upload(h, (uint16_t **)&ly.wx, wx16.data(), wx16.size() * 2, st, "input weights")
                      : upload(h, (float **)&ly.wx, wx32.data(), wx32.size() * 4, st, "input weights");
        if (rc == LSTM_OK && h->csr_dense_proj)
            rc = upload(h, (uint16_t **)&ly.wx, wx16.data(), wx16.size() * 2, st, "input weights (dense copy)");
        if (rc == LSTM_OK && csr) {
            rc = upload(h, &ly.wx_rowptr, px_rowptr.data(), px_rowptr.size() * sizeof(int), st, "input CSR offsets");
            if (rc == LSTM_OK) rc = upload(h, &ly.wx_ent, px_ent.data(), px_ent.size() * sizeof(CsrEntry), st, "input CSR entries");
        }
        if (rc == LSTM_OK && cudaStreamSynchronize(st) != cudaSuccess)
            rc = fail(h, LSTM_ERR_CUDA, "upload failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (rc) return bail(rc);

    if (h->use_csr_reg) {
        // one slot count for the whole handle: the longest lane list of any matrix, rounded up to a built size
        const int slots = recur_csr_reg_slots(std::max(h->csr_slots, 1), h->csr_nw);
        if (slots == 0) h->use_csr_reg = false;            // lists too long for registers: the shared-memory kernel runs
        if (!h->use_csr_reg) h->csr_fuse_ok = false;
        h->csr_slots = slots;
        for (int l = 0; l < layers && rc == LSTM_OK; ++l)
            for (int d = 0; d < D && rc == LSTM_OK; ++d) {
                Layer &ly = h->layers[l];
                if (h->use_csr_reg) {
                    long long conflicts = 0;
                    const std::vector<unsigned> packed = csr_pack_slots(ly.csr_lists[d], h->ncta_dir, h->csr_nw, slots, h->csr_kspan, &conflicts);
                    h->csr_conflicts = std::max(h->csr_conflicts, conflicts);
                    rc = upload(h, &ly.csr_reg_ent[d], packed.data(), packed.size() * 4, st, "sparse recurrent entries");
                    if (rc == LSTM_OK) rc = upload(h, &ly.csr_reg_rows[d], ly.csr_lists[d].rows.data(), ly.csr_lists[d].rows.size() * 4, st, "sparse recurrent rows");
                    if (rc == LSTM_OK) cudaStreamSynchronize(st);
                    cudaFree(ly.wh_ptr[d]); cudaFree(ly.wh_ent[d]);       // the shared-memory kernel's copy is not needed
                    ly.wh_ptr[d] = nullptr; ly.wh_ent[d] = nullptr;
                }
                ly.csr_lists[d] = CsrLaneLists();
            }
        if (rc) return bail(rc);
    }

    // workspace
    const size_t Mmax = (size_t)max_T * max_B;
    const size_t N = (size_t)D * 4 * H;
    h->G_cap = std::max(Mmax * N, std::min<size_t>(Mmax, 256) * N * n_split_cap());
    rc = dev_alloc(h, &h->G, h->G_cap * 4, false, st, "projection workspace");
    if (rc == LSTM_OK && h->use_tc) {
        h->ld0 = round_up(in_dim, 8);
        rc = dev_alloc(h, &h->xb0, 2 * Mmax * h->ld0 * 2, true, st, "bf16 input staging");
        if (rc == LSTM_OK && layers > 1) {
            h->ldn = round_up(D * H, 8);
            for (int i = 0; i < 2 && rc == LSTM_OK; ++i) rc = dev_alloc(h, &h->xbn[i], 2 * Mmax * h->ldn * 2, true, st, "bf16 layer activations");
        }
    }
    if (rc == LSTM_OK && layers > 1)
        for (int i = 0; i < 2 && rc == LSTM_OK; ++i) rc = dev_alloc(h, &h->ybuf[i], Mmax * D * H * 4, false, st, "layer activations");
    h->xch_words = (size_t)D * 2 * max_B * H;
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->xch, h->xch_words * 8, true, st, "exchange buffer");
    if (rc == LSTM_OK && h->use_tcb) {
        rc = dev_alloc(h, &h->hplanes, (size_t)D * 2 * kTcPlaneRows * h->tcb_ldh * 2, true, st, "h planes");
        if (rc == LSTM_OK) rc = dev_alloc(h, &h->tcb_flags, (size_t)D * h->ncta_dir * sizeof(unsigned), true, st, "stamps");
    }
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->status_dev, sizeof(int), true, st, "status word");
    if (rc == LSTM_OK && h->use_wave) {
        h->wave_xch_words = (size_t)layers * max_T * std::min(max_B, 4) * H;
        rc = dev_alloc(h, &h->wave_xch, h->wave_xch_words * 8, true, st, "wavefront exchange buffer");
        if (rc == LSTM_OK && recur_wave_prepare(h->wave_mt, h->wave_nkr, h->smem_optin - 64) != cudaSuccess)
            rc = fail(h, LSTM_ERR_CUDA, "wavefront kernel set-up failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (rc == LSTM_OK) {
        cudaError_t e = h->use_csr_reg ? recur_csr_reg_prepare(h->csr_slots, h->csr_nw, h->smem_optin - 64)
                            : csr ? recur_csr_prepare(h->smem_optin - 64)
                            : h->use_mma ? recur_mma_prepare(h->mma_mt, h->mma_nkr, h->mma_nw, h->smem_optin - 64)
                                         : recur_dense_prepare(h->smem_optin - 64);
        if (e == cudaSuccess && h->use_tc) e = proj_tc_prepare();
        if (e == cudaSuccess && csr) e = proj_csr_prepare(h->smem_optin - 64);
        if (e == cudaSuccess && h->use_tcb) e = recur_tc_prepare(h->smem_optin - kTcStaticSmem);
        if (e != cudaSuccess) rc = fail(h, LSTM_ERR_CUDA, "kernel set-up failed: %s", cudaGetErrorString(e));
    }
    if (rc == LSTM_OK && cudaStreamSynchronize(st) != cudaSuccess)
        rc = fail(h, LSTM_ERR_CUDA, "workspace set-up failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (rc) return bail(rc);
    *out = h;
    return LSTM_OK;
}

int lstm_create(lstm_handle **out, int layers, int in_dim, int hidden, int bidir, int dtype,
                const lstm_weights *w, int exec_mode, int max_T, int max_B, void *cuda_stream)
{
    return create_impl(out, layers, in_dim, hidden, bidir, dtype, w, exec_mode, max_T, max_B, cuda_stream, true);
}

// Row/column-pruned stacks (Section 4.2, Algorithm 1).  A hidden unit is REMOVED when nothing reads it and it
// reads nothing: its four gate rows are zero in Wx and Wh, its column of Wh is zero, and (below the last layer)
// its column of every next-layer Wx is zero.  When at least one unit per (layer, direction) can go, an inner
// handle is created over the surviving units (one common width Hc = the largest number of survivors; a matrix
// with more removable units keeps some of them) and *out becomes a thin handle that moves states and outputs
// between the two widths.  *done = false: nothing to compact, the caller creates the handle as usual.
static int try_compaction(lstm_handle **out, int layers, int in_dim, int hidden, int bidir, int dtype,
                          const lstm_weights *w, int exec_mode, int max_T, int max_B, void *cuda_stream, bool *done)
{
    *done = false;
    const int L = layers, D = bidir ? 2 : 1, H = hidden;
    if (H < 2) return LSTM_OK;
    std::vector<std::vector<float>> wx(L * D), wh(L * D), bs(L * D);
    std::vector<std::vector<char>> rows_zero(L * D);
    char name[64];
    // pass 1: units with four zero gate rows; most models have none, and then nothing else is looked at
    bool any = false;
    for (int ld = 0; ld < L * D; ++ld) {
        const int in_l = ld < D ? in_dim : D * H;
        snprintf(name, sizeof name, "wx[%d]", ld);
        int rc = matrix_to_dense(nullptr, 4 * H, in_l, w[ld].wx, w[ld].mask_x, w[ld].wx_rowptr, w[ld].wx_col, w[ld].wx_val, wx[ld], name);
        if (rc) return rc;
        snprintf(name, sizeof name, "wh[%d]", ld);
        rc = matrix_to_dense(nullptr, 4 * H, H, w[ld].wh, w[ld].mask_h, w[ld].wh_rowptr, w[ld].wh_col, w[ld].wh_val, wh[ld], name);
        if (rc) return rc;
        rows_zero[ld].assign(H, 1);
        int count = 0;
        for (int j = 0; j < H; ++j) {
            bool zero = true;
            for (int q = 0; q < 4 && zero; ++q) {
                const float *rx = wx[ld].data() + (size_t)(q * H + j) * in_l, *rh = wh[ld].data() + (size_t)(q * H + j) * H;
                for (int k = 0; k < in_l && zero; ++k) zero = rx[k] == 0.0f;
                for (int k = 0; k < H && zero; ++k) zero = rh[k] == 0.0f;
            }
            rows_zero[ld][j] = zero;
            count += zero;
        }
        if (count == 0) return LSTM_OK;                 // this matrix keeps all H units: the common width stays H
        any = true;
    }
    if (!any) return LSTM_OK;
    // pass 2: of those, the units nobody reads
    std::vector<std::vector<int>> keep(L * D), gone(L * D);
    int Hc = 1;
    for (int ld = 0; ld < L * D; ++ld) {
        const int l = ld / D, d = ld % D;
        std::vector<char> removable(rows_zero[ld]);
        for (int j = 0; j < H; ++j) {
            if (!removable[j]) continue;
            bool unread = true;
            for (int r = 0; r < 4 * H && unread; ++r) unread = wh[ld][(size_t)r * H + j] == 0.0f;
            if (l + 1 < L)
                for (int d2 = 0; d2 < D && unread; ++d2) {
                    const std::vector<float> &nx = wx[(l + 1) * D + d2];
                    for (int r = 0; r < 4 * H && unread; ++r) unread = nx[(size_t)r * (D * H) + (size_t)d * H + j] == 0.0f;
                }
            removable[j] = unread;
        }
        for (int j = 0; j < H; ++j) (removable[j] ? gone[ld] : keep[ld]).push_back(j);
        Hc = std::max(Hc, (int)keep[ld].size());
    }
    if (Hc >= H) return LSTM_OK;
    // one width for the whole stack: matrices with fewer survivors keep some removable units
    for (int ld = 0; ld < L * D; ++ld) {
        while ((int)keep[ld].size() < Hc) { keep[ld].push_back(gone[ld].back()); gone[ld].pop_back(); }
        std::sort(keep[ld].begin(), keep[ld].end());
        std::sort(gone[ld].begin(), gone[ld].end());
    }
    // the compact model's weights (dense, zeros written in)
    std::vector<std::vector<float>> cwx(L * D), cwh(L * D), cb(L * D);
    std::vector<lstm_weights> cw(L * D);
    std::vector<int> cmap((size_t)L * D * Hc), rem_idx;
    std::vector<float> rem_bias;
    for (int ld = 0; ld < L * D; ++ld) {
        const int l = ld / D;
        const int in_l = l == 0 ? in_dim : D * H, cin_l = l == 0 ? in_dim : D * Hc;
        HostView bv;
        if (!host_view(w[ld].b, sizeof(float) * 4 * H, bv)) return fail(nullptr, LSTM_ERR_CUDA, "reading bias");
        const float *b = (const float *)bv.ptr;
        cwx[ld].assign((size_t)4 * Hc * cin_l, 0.0f);
        cwh[ld].assign((size_t)4 * Hc * Hc, 0.0f);
        cb[ld].assign((size_t)4 * Hc, 0.0f);
        for (int jc = 0; jc < Hc; ++jc) cmap[(size_t)ld * Hc + jc] = keep[ld][jc];
        for (int q = 0; q < 4; ++q)
            for (int jc = 0; jc < Hc; ++jc) {
                const int j = keep[ld][jc];
                const float *rx = wx[ld].data() + (size_t)(q * H + j) * in_l, *rh = wh[ld].data() + (size_t)(q * H + j) * H;
                float *dx = cwx[ld].data() + (size_t)(q * Hc + jc) * cin_l, *dh = cwh[ld].data() + (size_t)(q * Hc + jc) * Hc;
                if (l == 0) memcpy(dx, rx, sizeof(float) * in_dim);
                else
                    for (int d2 = 0; d2 < D; ++d2) {
                        const std::vector<int> &kp = keep[(l - 1) * D + d2];
                        for (int kc = 0; kc < Hc; ++kc) dx[(size_t)d2 * Hc + kc] = rx[(size_t)d2 * H + kp[kc]];
                    }
                for (int kc = 0; kc < Hc; ++kc) dh[kc] = rh[keep[ld][kc]];
                if (b) cb[ld][(size_t)q * Hc + jc] = b[q * H + j];
            }
        for (int j : gone[ld]) {
            rem_idx.push_back(ld); rem_idx.push_back(j);
            for (int q = 0; q < 4; ++q) rem_bias.push_back(b ? b[q * H + j] : 0.0f);
        }
        memset(&cw[ld], 0, sizeof(lstm_weights));
        cw[ld].wx = cwx[ld].data(); cw[ld].wh = cwh[ld].data(); cw[ld].b = cb[ld].data();
        wx[ld] = std::vector<float>(); wh[ld] = std::vector<float>();
    }
    lstm_handle *inner = nullptr;
    int rc = create_impl(&inner, layers, in_dim, Hc, bidir, dtype, cw.data(), exec_mode, max_T, max_B, cuda_stream, false);
    if (rc != LSTM_OK) return rc;
    lstm_handle *h = new (std::nothrow) lstm_handle;
    if (!h) { lstm_destroy(inner); return fail(nullptr, LSTM_ERR_NOMEM, "host allocation failed"); }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->L = L; h->D = D; h->in_dim = in_dim; h->H = H; h->dtype = dtype; h->exec_mode = exec_mode;
    h->max_T = max_T; h->max_B = max_B; h->device = inner->device; h->sm_count = inner->sm_count; h->smem_optin = inner->smem_optin;
    h->last_stream = st;
    h->inner = inner; h->Hc = Hc; h->n_removed = (int)(rem_idx.size() / 2);
    const size_t sn = (size_t)L * D * max_B * Hc;
    rc = upload(h, &h->cmap, cmap.data(), cmap.size() * sizeof(int), st, "unit map");
    if (rc == LSTM_OK) rc = upload(h, &h->rem_idx, rem_idx.data(), rem_idx.size() * sizeof(int), st, "removed units");
    if (rc == LSTM_OK) rc = upload(h, &h->rem_bias, rem_bias.data(), rem_bias.size() * sizeof(float), st, "removed units' bias");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->ch0, sn * 4, false, st, "compact h0");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->cc0, sn * 4, false, st, "compact c0");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->chT, sn * 4, false, st, "compact hT");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->ccT, sn * 4, false, st, "compact cT");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->cy, (size_t)max_T * max_B * D * Hc * 4, false, st, "compact y");
    if (rc == LSTM_OK && cudaStreamSynchronize(st) != cudaSuccess)
        rc = fail(h, LSTM_ERR_CUDA, "upload failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (rc != LSTM_OK) { g_create_error = h->err; lstm_destroy(h); return rc; }
    *out = h;
    *done = true;
    return LSTM_OK;
}

int hlstm_create(lstm_handle **out, int layers, int in_dim, int hidden, int gate_hidden, int bidir, int dtype,
                 const hlstm_weights *w, int max_T, int max_B, void *cuda_stream)
{
    if (!out) return fail(nullptr, LSTM_ERR_INVALID, "out is NULL");
    *out = nullptr;
    if (layers < 1 || in_dim < 1 || hidden < 1 || gate_hidden < 1 || (bidir != 0 && bidir != 1) || !w || max_T < 1 || max_B < 1)
        return fail(nullptr, LSTM_ERR_INVALID, "bad argument: layers=%d in_dim=%d hidden=%d gate_hidden=%d bidir=%d max_T=%d max_B=%d w=%p",
                    layers, in_dim, hidden, gate_hidden, bidir, max_T, max_B, (const void *)w);
    if (dtype != LSTM_F32 && dtype != LSTM_BF16W_F32S) return fail(nullptr, LSTM_ERR_INVALID, "unknown dtype %d", dtype);
    if (dtype != LSTM_BF16W_F32S) return fail(nullptr, LSTM_ERR_UNSUPPORTED, "the H-LSTM cell is served with bf16 weights only");
    if (hidden >= 65536 || gate_hidden >= 65536) return fail(nullptr, LSTM_ERR_UNSUPPORTED, "hidden widths must be < 65536");
    if ((long long)max_T * max_B > (1LL << 30)) return fail(nullptr, LSTM_ERR_UNSUPPORTED, "max_T*max_B too large");
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        const char *m = cudaGetErrorString(cudaGetLastError());
        return fail(nullptr, LSTM_ERR_CUDA, "no usable CUDA device: %s", m);
    }
    if (prop.major != 10) return fail(nullptr, LSTM_ERR_CUDA, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
    int coop = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (!coop) return fail(nullptr, LSTM_ERR_CUDA, "device does not support cooperative launch");

    lstm_handle *h = new (std::nothrow) lstm_handle;
    if (!h) return fail(nullptr, LSTM_ERR_NOMEM, "host allocation failed");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int H = hidden, Hh = gate_hidden, D = bidir ? 2 : 1;
    h->L = layers; h->D = D; h->in_dim = in_dim; h->H = H; h->Hh = Hh; h->dtype = dtype;
    h->exec_mode = LSTM_DENSE; h->max_T = max_T; h->max_B = max_B; h->device = dev;
    h->sm_count = prop.multiProcessorCount;
    h->smem_optin = (int)prop.sharedMemPerBlockOptin;
    h->last_stream = st;
    h->Hp8 = round_up(H, 8); h->Hs = round_up(H, 256);
    h->ncta_dir = std::max(1, std::min(h->sm_count / D, std::max(H, Hh)));   // a CTA may own no unit of the narrower side
    h->upc = (H + h->ncta_dir - 1) / h->ncta_dir;
    h->threads = 512;
    h->use_tc = true;
    h->layers.resize(layers);
    if (const char *env = getenv("LSTM_B200_SPIN_LIMIT")) { long long v = atoll(env); if (v > 0) h->spin_limit = v; }
    h->spin_limit_default = h->spin_limit;
    auto bail = [&](int code) { g_create_error = h->err; free_all(h); delete h; return code; };

    // tiling: row tiles cover 4 x (units per CTA) of both passes; pass 1 keeps up to nkr column tiles per
    // warp in registers, the rest and all of pass 2 in shared memory
    {
        const int upch = (Hh + h->ncta_dir - 1) / h->ncta_dir;
        const int mt = (4 * std::max(h->upc, upch) + 15) / 16;
        const int nk1 = (H + 15) / 16, nk2 = (Hh + 15) / 16;
        const int nw = (nk1 <= 32 && nk2 <= 32 && std::max(h->upc, upch) <= 8) ? 8 : 16;
        const int need1 = (nk1 + nw - 1) / nw, need2 = (nk2 + nw - 1) / nw;
        bool ok = mt <= 4 && std::max(h->upc, upch) <= nw;
        int nkr = 0;
        if (ok) {
            const int cap = (nw == 16 ? kMmaTileCap16 : kMmaTileCap8) / mt;
            for (int c = 2; c <= 8; c += 2)
                if (c <= cap && (nkr == 0 || nkr < need1)) nkr = c;
            ok = nkr > 0 && recur_mma_shape_ok(mt, nkr, nw);
        }
        const int nks1 = ok && need1 > nkr ? need1 - nkr : 0;
        if (ok) ok = hlstm_mma_smem_bytes(mt, nkr, nw, nks1, need2, h->upc, max_B) <= (size_t)h->smem_optin - 64;
        if (!ok) {
            fail(h, LSTM_ERR_UNSUPPORTED, "hidden=%d gate_hidden=%d max_B=%d: the per-CTA slices do not fit registers and shared memory", H, Hh, max_B);
            return bail(LSTM_ERR_UNSUPPORTED);
        }
        h->use_mma = true;
        h->mma_mt = mt; h->mma_nkr = nkr; h->mma_nks = nks1; h->mma_nw = nw; h->hl_nkw2 = need2;
    }

    int rc = LSTM_OK;
    for (int l = 0; l < layers && rc == LSTM_OK; ++l) {
        Layer &ly = h->layers[l];
        ly.in_l = l == 0 ? in_dim : D * H;
        ly.ldk = round_up(ly.in_l, 8);
        const int N = D * 4 * Hh;
        std::vector<float> bias_p((size_t)N, 0.0f), bias_o((size_t)D * 4 * H, 0.0f);
        std::vector<uint16_t> wx16((size_t)N * ly.ldk, 0);
        for (int d = 0; d < D && rc == LSTM_OK; ++d) {
            const hlstm_weights &src = w[l * D + d];
            if (!src.ux || !src.uh || !src.w) { rc = fail(h, LSTM_ERR_INVALID, "ux, uh and w must be given (layer %d, dir %d)", l, d); break; }
            HostView v_ux, v_uh, v_w, v_a, v_b;
            if (!host_view(src.ux, sizeof(float) * 4 * Hh * ly.in_l, v_ux) || !host_view(src.uh, sizeof(float) * 4 * Hh * H, v_uh) ||
                !host_view(src.w, sizeof(float) * 4 * H * Hh, v_w) || !host_view(src.a, sizeof(float) * 4 * Hh, v_a) ||
                !host_view(src.b, sizeof(float) * 4 * H, v_b)) { rc = fail(h, LSTM_ERR_CUDA, "reading weights"); break; }
            const float *ux = (const float *)v_ux.ptr, *uh = (const float *)v_uh.ptr, *ww = (const float *)v_w.ptr;
            const float *ba = (const float *)v_a.ptr, *bb = (const float *)v_b.ptr;
            // keep-masks: the masked copies replace the caller's matrices
            std::vector<float> ux_m, uh_m, w_m;
            auto masked = [&](const float *&m, const unsigned char *mask, size_t n, std::vector<float> &store) -> bool {
                if (!mask) return true;
                HostView v;
                if (!host_view(mask, n, v)) return false;
                const unsigned char *mk = (const unsigned char *)v.ptr;
                store.resize(n);
                for (size_t i = 0; i < n; ++i) store[i] = mk[i] ? m[i] : 0.0f;
                m = store.data();
                return true;
            };
            if (!masked(ux, src.mask_ux, (size_t)4 * Hh * ly.in_l, ux_m) || !masked(uh, src.mask_uh, (size_t)4 * Hh * H, uh_m) ||
                !masked(ww, src.mask_w, (size_t)4 * H * Hh, w_m)) { rc = fail(h, LSTM_ERR_CUDA, "reading masks"); break; }
            for (int q = 0; q < 4; ++q) {
                for (int m = 0; m < Hh; ++m) {
                    const size_t prow = (size_t)d * 4 * Hh + (size_t)m * 4 + q;           // unit-major, gates adjacent
                    if (ba) bias_p[prow] = ba[q * Hh + m];
                    const float *srow = ux + (size_t)(q * Hh + m) * ly.in_l;
                    for (int k = 0; k < ly.in_l; ++k) wx16[prow * ly.ldk + k] = f32_to_bf16_rne(srow[k]);
                }
                if (bb) for (int j = 0; j < H; ++j) bias_o[(size_t)d * 4 * H + (size_t)j * 4 + q] = bb[q * H + j];
            }
            const int NW = h->mma_nw;
            std::vector<uint32_t> f1 = pack_fragments(uh, Hh, H, h->ncta_dir, NW, h->mma_nkr + h->mma_nks, h->mma_mt);
            std::vector<uint32_t> f2 = pack_fragments(ww, H, Hh, h->ncta_dir, NW, h->hl_nkw2, h->mma_mt);
            rc = upload(h, (uint32_t **)&ly.wfrag[d], f1.data(), f1.size() * 4, st, "hidden-layer recurrent fragments");
            if (rc == LSTM_OK) rc = upload(h, (uint32_t **)&ly.frag2[d], f2.data(), f2.size() * 4, st, "gate output fragments");
            if (rc == LSTM_OK) cudaStreamSynchronize(st);
        }
        if (rc) break;
        rc = upload(h, &ly.bias, bias_p.data(), bias_p.size() * 4, st, "hidden-layer bias");
        if (rc == LSTM_OK) rc = upload(h, &ly.bias_out, bias_o.data(), bias_o.size() * 4, st, "gate bias");
        if (rc == LSTM_OK) rc = upload(h, (uint16_t **)&ly.wx, wx16.data(), wx16.size() * 2, st, "input weights");
        if (rc == LSTM_OK && cudaStreamSynchronize(st) != cudaSuccess)
            rc = fail(h, LSTM_ERR_CUDA, "upload failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (rc) return bail(rc);

    const size_t Mmax = (size_t)max_T * max_B;
    const size_t N = (size_t)D * 4 * Hh;
    h->G_cap = std::max(Mmax * N, std::min<size_t>(Mmax, 256) * N * n_split_cap());
    rc = dev_alloc(h, &h->G, h->G_cap * 4, false, st, "projection workspace");
    h->ld0 = round_up(in_dim, 8);
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->xb0, 2 * Mmax * h->ld0 * 2, true, st, "bf16 input staging");
    if (layers > 1) {
        h->ldn = round_up(D * H, 8);
        for (int i = 0; i < 2 && rc == LSTM_OK; ++i) rc = dev_alloc(h, &h->xbn[i], 2 * Mmax * h->ldn * 2, true, st, "bf16 layer activations");
        for (int i = 0; i < 2 && rc == LSTM_OK; ++i) rc = dev_alloc(h, &h->ybuf[i], Mmax * D * H * 4, false, st, "layer activations");
    }
    h->xch_words = (size_t)D * 2 * max_B * H;
    h->rxch_words = (size_t)D * 2 * max_B * 4 * Hh;
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->xch, h->xch_words * 8, true, st, "exchange buffer");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->rxch, h->rxch_words * 8, true, st, "hidden-layer exchange buffer");
    if (rc == LSTM_OK) rc = dev_alloc(h, &h->status_dev, sizeof(int), true, st, "status word");
    if (rc == LSTM_OK) {
        cudaError_t e = hlstm_mma_prepare(h->mma_mt, h->mma_nkr, h->mma_nw, h->smem_optin - 64);
        if (e == cudaSuccess) e = proj_tc_prepare();
        if (e != cudaSuccess) rc = fail(h, LSTM_ERR_CUDA, "kernel set-up failed: %s", cudaGetErrorString(e));
    }
    if (rc == LSTM_OK && cudaStreamSynchronize(st) != cudaSuccess)
        rc = fail(h, LSTM_ERR_CUDA, "workspace set-up failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (rc) return bail(rc);
    *out = h;
    return LSTM_OK;
}

static int record(lstm_handle *h, int kind, cudaStream_t st)
{
    if (!h->prof) return 0;
    if (h->ev_used >= (int)h->ev.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return 1;
        h->ev.push_back(e);
        h->ev_kind.push_back(kind);
    }
    h->ev_kind[h->ev_used] = kind;
    return cudaEventRecord(h->ev[h->ev_used++], st) != cudaSuccess;
}

// Input staging (layer 0, tensor-core path) and projection of layer l for M rows into h->G; *nsplit receives
// the number of split-K planes written.  x: the call's input (layer 0 only), Xf: fp32 activations of the layer.
static int run_projection(lstm_handle *h, int l, const float *x, const float *Xf, int M, int N, int *nsplit_out, cudaStream_t st)
{
    Layer &ly = h->layers[l];
    const bool bf16 = h->dtype == LSTM_BF16W_F32S;
    const bool csr = h->exec_mode == LSTM_CSR;
    cudaError_t e = cudaSuccess;
    int nsplit = 1;
    // ---- input staging + projection
    if (csr && !h->csr_dense_proj) {
        if (record(h, LSTM_K_PROJ, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        e = launch_proj_csr(Xf, ly.wx_rowptr, ly.wx_ent, ly.bias, h->G, M, N, ly.in_l, !bf16, st);
        ++h->last_launches;
        if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
    } else if (h->use_tc) {
        __nv_bfloat16 *xb = l == 0 ? h->xb0 : h->xbn[(l - 1) & 1];
        if (l == 0) {
            if (record(h, LSTM_K_STAGE, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            e = launch_stage_bf16(x, xb, (long long)h->max_T * h->max_B * h->ld0, M, h->in_dim, h->ld0, st);
            ++h->last_launches;
            if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "staging launch failed: %s", cudaGetErrorString(e));
        }
        if (ly.plan_M != M) {
            char msg[256];
            const long long plane = (long long)h->max_T * h->max_B * ly.ldk;
            if (proj_tc_plan(&ly.plan, (const __nv_bfloat16 *)ly.wx, xb, xb + plane, M, N, ly.in_l, ly.ldk, h->sm_count, msg, sizeof msg))
                return fail(h, LSTM_ERR_CUDA, "tensor-core projection plan failed: %s", msg);
            ly.plan_M = M;
        }
        nsplit = ly.plan.nsplit;
        if ((size_t)nsplit * M * N > h->G_cap) return fail(h, LSTM_ERR_CUDA, "internal: projection workspace too small");
        if (record(h, LSTM_K_PROJ, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        e = launch_proj_tc(ly.plan, ly.bias, h->G, h->status_dev, st);
        ++h->last_launches;
        if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
    } else {
        if (record(h, LSTM_K_PROJ, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        e = launch_proj_simt(Xf, ly.wx, bf16, ly.ldk, ly.bias, h->G, M, N, ly.in_l, st);
        ++h->last_launches;
        if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
    }
    if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "projection launch failed (layer %d): %s", l, cudaGetErrorString(e));
    *nsplit_out = nsplit;
    return LSTM_OK;
}

int lstm_forward(lstm_handle *h, const float *x, int T, int B, const float *h0, const float *c0,
                 float *y, float *hT, float *cT, void *cuda_stream)
{
    if (!h) return LSTM_ERR_INVALID;
    if (T < 0 || B < 0 || T > h->max_T || B > h->max_B)
        return fail(h, LSTM_ERR_INVALID, "T=%d B=%d outside [0,%d] x [0,%d]", T, B, h->max_T, h->max_B);
    if (const int drc = check_device(h)) return drc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->last_stream = st;
    const int L = h->L, D = h->D, H = h->H;
    const size_t state_n = (size_t)L * D * B * H;
    h->ev_used = 0;
    h->last_launches = 0;
    if (T == 0 || B == 0) {
        if (B > 0 && state_n) {
            for (int i = 0; i < 2; ++i) {
                float *dst = i ? cT : hT;
                const float *src = i ? c0 : h0;
                if (!dst) continue;
                cudaError_t e = src ? cudaMemcpyAsync(dst, src, state_n * 4, cudaMemcpyDeviceToDevice, st)
                                    : cudaMemsetAsync(dst, 0, state_n * 4, st);
                if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "state copy failed: %s", cudaGetErrorString(e));
            }
        }
        return LSTM_OK;
    }
    if (!x || !y) return fail(h, LSTM_ERR_INVALID, "x and y must not be NULL");

    if (h->inner) {
        // row/column-pruned stack: states to the compact width, the pass over the surviving units, outputs back
        CompactArgs ca;
        memset(&ca, 0, sizeof ca);
        ca.L = L; ca.D = D; ca.H = H; ca.Hc = h->Hc; ca.T = T; ca.B = B;
        ca.cmap = h->cmap; ca.n_removed = h->n_removed; ca.rem_idx = h->rem_idx; ca.rem_bias = h->rem_bias;
        ca.h0 = h0; ca.c0 = c0; ca.h0c = h->ch0; ca.c0c = h->cc0;
        ca.yc = h->cy; ca.hTc = h->chT; ca.cTc = h->ccT; ca.y = y; ca.hT = hT; ca.cT = cT;
        int extra = 0;
        if (h0 || c0) {
            const cudaError_t ge = launch_compact_gather(ca, st);
            if (ge != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "state gather failed: %s", cudaGetErrorString(ge));
            ++extra;
        }
        const int irc = lstm_forward(h->inner, x, T, B, h0 ? h->ch0 : nullptr, c0 ? h->cc0 : nullptr, h->cy,
                                     h->chT, h->ccT, cuda_stream);
        if (irc != LSTM_OK) return fail(h, irc, "%s", h->inner->err.c_str());
        const cudaError_t se = launch_compact_scatter(ca, st);
        if (se != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "output scatter failed: %s", cudaGetErrorString(se));
        h->last_launches = h->inner->last_launches + extra + 1;
        return LSTM_OK;
    }

    const int M = T * B;
    const bool bf16 = h->dtype == LSTM_BF16W_F32S;
    const bool csr = h->exec_mode == LSTM_CSR;
    cudaError_t e = cudaSuccess;

    // stamps of the exchange words must stay unique: restart from a cleared buffer before wrapping
    if ((unsigned long long)h->stamp_next + (unsigned long long)L * D * ((unsigned long long)T + 1ull) + 2ull >= 0xffffffffull) {
        if (cudaMemsetAsync(h->xch, 0, h->xch_words * 8, st) != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "exchange reset failed");
        if (h->rxch && cudaMemsetAsync(h->rxch, 0, h->rxch_words * 8, st) != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "exchange reset failed");
        if (h->tcb_flags && cudaMemsetAsync(h->tcb_flags, 0, (size_t)D * h->ncta_dir * sizeof(unsigned), st) != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "exchange reset failed");
        if (h->wave_xch && cudaMemsetAsync(h->wave_xch, 0, h->wave_xch_words * 8, st) != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "exchange reset failed");
        h->stamp_next = 1;
    }

    if (h->use_wave && B <= 4 && !h->probe) {          // (the probe builds exist for the per-layer kernels)
        // all layers in one launch: layer 0's projection for all timesteps, then the wavefront kernel
        int nsplit = 1;
        { const int prc = run_projection(h, 0, x, x, M, D * 4 * H, &nsplit, st); if (prc != LSTM_OK) return prc; }
        RecurWaveArgs m;
        memset(&m, 0, sizeof m);
        m.L = L; m.H = H; m.B = B; m.T = T; m.ncta_layer = h->wave_ncta; m.nsplit = nsplit;
        for (int l = 0; l < L; ++l) { m.nkw[l] = h->wave_nkw[l]; m.wfrag[l] = h->wave_frag[l]; m.bias[l] = h->layers[l].bias; }
        m.nkw_max = h->wave_nkw_max;
        m.stamp_base = h->stamp_next;
        h->stamp_next += (unsigned)T + 1u;
        m.spin_limit = h->spin_limit;
        m.withhold_cta = h->withhold_cta;
        m.G = h->G;
        m.g_split_stride = (long long)M * 4 * H;
        m.h0 = h0; m.c0 = c0; m.hT = hT; m.cT = cT; m.y = y;
        m.xch = h->wave_xch;
        m.status = h->status_dev;
        const size_t smem = recur_wave_smem_bytes(h->wave_mt, h->wave_nkr, h->wave_nkw_max, h->wave_upc, B);
        if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        e = launch_recur_wave(m, h->wave_mt, h->wave_nkr, smem, st);
        ++h->last_launches;
        if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "wavefront launch failed: %s", cudaGetErrorString(e));
        return LSTM_OK;
    }

    for (int l = 0; l < L; ++l) {
        Layer &ly = h->layers[l];
        const float *Xf = l == 0 ? x : h->ybuf[(l - 1) & 1];
        const int N = D * 4 * (h->Hh ? h->Hh : H);      // H-LSTM: the projection feeds the hidden layers
        int nsplit = 1;
        // ---- input staging + projection (a single short sequence on the register-resident kernel computes its
        // projection inside that kernel's prologue instead: two launches and one round trip of G fewer per layer)
        const bool fuse = (h->fuse_ok || (h->csr_fuse_ok && h->use_csr_reg)) && !h->Hh && B == 1 && T <= kFuseMaxT && !h->probe &&
                          ly.xfrag[0] != nullptr;
        if (!fuse) { const int prc = run_projection(h, l, l == 0 ? x : nullptr, Xf, M, N, &nsplit, st); if (prc != LSTM_OK) return prc; }

        // ---- recurrence: all directions in one launch, or one launch per direction
        const int npass = h->seq_dirs ? D : 1;
        for (int pass = 0; pass < npass; ++pass) {
        if (h->Hh) {
            HlstmArgs m;
            memset(&m, 0, sizeof m);
            m.dir0 = h->seq_dirs ? pass : 0; m.ndirs = h->seq_dirs ? 1 : D;
            m.H = H; m.Hh = h->Hh; m.B = B; m.T = T; m.D = D; m.ncta_dir = h->ncta_dir; m.nsplit = nsplit;
            m.nks1 = h->mma_nks; m.nkw2 = h->hl_nkw2;
            m.stamp_base = h->stamp_next;
            h->stamp_next += (unsigned)T + 1u;
            m.spin_limit = h->spin_limit;
            m.withhold_cta = h->withhold_cta;
            for (int d = 0; d < D; ++d) { m.frag1[d] = ly.wfrag[d]; m.frag2[d] = ly.frag2[d]; }
            m.G = h->G;
            m.g_split_stride = (long long)M * N;
            m.bias_out = ly.bias_out;
            const size_t so = (size_t)l * D * B * H;
            m.h0 = h0 ? h0 + so : nullptr; m.c0 = c0 ? c0 + so : nullptr;
            m.hT = hT ? hT + so : nullptr; m.cT = cT ? cT + so : nullptr;
            m.y = l == L - 1 ? y : h->ybuf[l & 1];
            m.xb_next = l < L - 1 ? h->xbn[l & 1] : nullptr;
            m.xb_ld = h->ldn;
            m.xb_plane = (long long)h->max_T * h->max_B * h->ldn;
            m.xch = h->xch; m.rxch = h->rxch;
            m.status = h->status_dev;
            const size_t smem = hlstm_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->hl_nkw2, h->upc, B);
            if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            e = launch_hlstm_mma(m, h->mma_mt, h->mma_nkr, h->mma_nw, smem, st);
            ++h->last_launches;
            if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "recurrent launch failed (layer %d): %s", l, cudaGetErrorString(e));
            continue;
        }
        int tc_kbs = 0, tc_stages = 0;
        // the batched kernel serves this call if the operand ring for this batch fits beside the resident slice
        // (the plan made at create time covers up to 32 sequences; larger batches may not fit and then run as
        // passes of four on the kernels below)
        if (h->use_tcb && B > 4 && B <= kTcMaxBatch &&
            recur_tc_plan(h->tcb_RA, h->tcb_nkb, round_up(2 * B, 16), h->upc, B, (size_t)h->smem_optin - kTcStaticSmem, h->tcb_pair ? 1 : 0, &tc_kbs, &tc_stages)) {
            RecurTcArgs m;
            memset(&m, 0, sizeof m);
            m.dir0 = h->seq_dirs ? pass : 0; m.ndirs = h->seq_dirs ? 1 : D;
            m.H = H; m.B = B; m.T = T; m.D = D; m.ncta_dir = h->ncta_dir; m.nsplit = nsplit;
            m.RA = h->tcb_RA; m.nkb = h->tcb_nkb; m.N = round_up(2 * B, 16);
            m.pair = h->tcb_pair ? 1 : 0;
            m.kbs = tc_kbs; m.stages = tc_stages;
            {
                // issuing threads: as many as the smaller K share of a CTA allows, at most three
                const int nkb_min = m.pair ? m.nkb / 2 : m.nkb;
                int ni = nkb_min >= 3 ? 3 : nkb_min >= 2 ? 2 : 1;
                if (const char *e = getenv("LSTM_B200_TC_ISSUE")) {
                    const int want = atoi(e);
                    if (want >= 1 && want <= ni) ni = want;
                }
                m.nissue = ni;
                const int cols = ni * m.N;
                m.tmem_cols = cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
            }
            m.ldh = h->tcb_ldh;
            m.stamp_base = h->stamp_next;
            h->stamp_next += (unsigned)T + 1u;
            m.spin_limit = h->spin_limit;
            m.withhold_cta = h->withhold_cta;
            m.G = h->G;
            m.g_split_stride = (long long)M * N;
            const size_t so = (size_t)l * D * B * H;
            m.h0 = h0 ? h0 + so : nullptr; m.c0 = c0 ? c0 + so : nullptr;
            m.hT = hT ? hT + so : nullptr; m.cT = cT ? cT + so : nullptr;
            m.y = l == L - 1 ? y : h->ybuf[l & 1];
            m.xb_next = (l < L - 1 && h->use_tc) ? h->xbn[l & 1] : nullptr;
            m.xb_ld = h->ldn;
            m.xb_plane = (long long)h->max_T * h->max_B * h->ldn;
            m.hbuf = h->hplanes; m.flags = h->tcb_flags;
            m.status = h->status_dev;
            if (h->tcb_mapN != B) {
                if (!recur_tc_encode_planes(h->tmap_planes, h->hplanes, D, H, h->tcb_ldh, B))
                    return fail(h, LSTM_ERR_CUDA, "tensor map of the h planes could not be encoded");
                h->tcb_mapN = B;
            }
            const size_t smem = recur_tc_smem_bytes(m.RA, m.nkb, m.N, m.stages, m.kbs, h->upc, B, m.pair);
            if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            e = launch_recur_tc(ly.tmap_wtc, h->tmap_planes, m, smem, st);
            ++h->last_launches;
            if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "recurrent launch failed (layer %d): %s", l, cudaGetErrorString(e));
            continue;
        }
        if (h->use_csr_reg) {
            RecurCsrArgs m;
            memset(&m, 0, sizeof m);
            m.dir0 = h->seq_dirs ? pass : 0; m.ndirs = h->seq_dirs ? 1 : D;
            m.H = H; m.B = B; m.T = T; m.D = D; m.ncta_dir = h->ncta_dir; m.nsplit = nsplit;
            m.kspan = h->csr_kspan; m.mt = h->csr_mt;
            m.stamp_base = h->stamp_next;
            h->stamp_next += (unsigned)T + 1u;
            m.spin_limit = h->spin_limit;
            m.withhold_cta = h->withhold_cta;
            m.probe = B == 1 ? h->probe : 0;
            for (int d = 0; d < D; ++d) { m.ent[d] = ly.csr_reg_ent[d]; m.rows[d] = ly.csr_reg_rows[d]; }
            m.G = h->G;
            m.g_split_stride = (long long)M * N;
            const size_t so = (size_t)l * D * B * H;
            m.h0 = h0 ? h0 + so : nullptr; m.c0 = c0 ? c0 + so : nullptr;
            m.hT = hT ? hT + so : nullptr; m.cT = cT ? cT + so : nullptr;
            m.y = l == L - 1 ? y : h->ybuf[l & 1];
            m.xb_next = (l < L - 1 && h->use_tc && !fuse) ? h->xbn[l & 1] : nullptr;     // a fused next layer reads the fp32 activations
            m.xb_ld = h->ldn;
            m.xb_plane = (long long)h->max_T * h->max_B * h->ldn;
            m.xch = h->xch;
            m.status = h->status_dev;
            m.fuse = fuse ? 1 : 0;
            m.in_l = ly.in_l; m.nkw_x = ly.nkw_x; m.X = Xf; m.bias = ly.bias;
            m.gs_off = (int)recur_csr_reg_fuse_gs_offset(h->csr_nw, h->csr_kspan, h->csr_mt, h->upc);
            for (int d = 0; d < D; ++d) m.xfrag[d] = ly.xfrag[d];
            const size_t smem = fuse ? recur_csr_reg_fuse_smem_bytes(h->csr_nw, h->csr_kspan, h->csr_mt, h->upc)
                                     : recur_csr_reg_smem_bytes(h->csr_nw, h->csr_kspan, h->csr_mt, h->upc, B);
            if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            e = launch_recur_csr_reg(m, h->csr_slots, h->csr_nw, smem, st);
            ++h->last_launches;
            if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "recurrent launch failed (layer %d): %s", l, cudaGetErrorString(e));
            continue;
        }
        const RecurShape shp = recur_shape(h, B, l);
        if (h->use_mma) {
            RecurMmaArgs m;
            memset(&m, 0, sizeof m);
            m.dir0 = h->seq_dirs ? pass : 0; m.ndirs = h->seq_dirs ? 1 : D;
            m.H = H; m.B = B; m.T = T; m.D = D; m.ncta_dir = h->ncta_dir; m.nsplit = nsplit; m.nkw_smem = h->mma_nks; m.staged = shp.staged ? 1 : 0;
            m.stamp_base = h->stamp_next;
            h->stamp_next += (unsigned)T + 1u;
            m.spin_limit = h->spin_limit;
            m.withhold_cta = h->withhold_cta;
            m.probe = B == 1 ? h->probe : 0;
            m.fuse = fuse ? 1 : 0;
            m.in_l = ly.in_l; m.nkw_x = ly.nkw_x; m.X = Xf; m.bias = ly.bias;
            m.gs_off = (int)recur_mma_fuse_gs_offset(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->upc);
            for (int d = 0; d < D; ++d) { m.wfrag[d] = ly.wfrag[d]; m.xfrag[d] = ly.xfrag[d]; }
            m.G = h->G;
            m.g_split_stride = (long long)M * N;
            const size_t so = (size_t)l * D * B * H;
            m.h0 = h0 ? h0 + so : nullptr; m.c0 = c0 ? c0 + so : nullptr;
            m.hT = hT ? hT + so : nullptr; m.cT = cT ? cT + so : nullptr;
            m.y = l == L - 1 ? y : h->ybuf[l & 1];
            m.xb_next = (l < L - 1 && h->use_tc && !fuse) ? h->xbn[l & 1] : nullptr;     // a fused next layer reads the fp32 activations
            m.xb_ld = h->ldn;
            m.xb_plane = (long long)h->max_T * h->max_B * h->ldn;
            m.xch = h->xch;
            m.status = h->status_dev;
            if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            e = launch_recur_mma(m, h->mma_mt, h->mma_nkr, h->mma_nw, fuse ? recur_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->upc, 1, false, true) : shp.smem, st);
            ++h->last_launches;
            if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
            if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "recurrent launch failed (layer %d): %s", l, cudaGetErrorString(e));
            continue;
        }
        RecurArgs a;
        memset(&a, 0, sizeof a);
        a.dir0 = h->seq_dirs ? pass : 0; a.ndirs = h->seq_dirs ? 1 : D;
        a.H = H; a.Hp8 = h->Hp8; a.Hs = h->Hs; a.B = B; a.T = T; a.D = D;
        a.ncta_dir = h->ncta_dir; a.nsplit = nsplit; a.BT = shp.BT; a.w_smem_bytes = shp.w_smem_bytes; a.stage_all = shp.stage_all ? 1 : 0;
        a.stamp_base = h->stamp_next;
        h->stamp_next += (unsigned)T + 1u;
        a.spin_limit = h->spin_limit;
        a.withhold_cta = h->withhold_cta;
        for (int d = 0; d < D; ++d) { a.wh[d] = ly.wh[d]; a.csr_ptr[d] = ly.wh_ptr[d]; a.csr_ent[d] = ly.wh_ent[d]; }
        a.G = h->G;
        a.g_split_stride = (long long)M * N;
        const size_t soff = (size_t)l * D * B * H;
        a.h0 = h0 ? h0 + soff : nullptr; a.c0 = c0 ? c0 + soff : nullptr;
        a.hT = hT ? hT + soff : nullptr; a.cT = cT ? cT + soff : nullptr;
        a.y = l == L - 1 ? y : h->ybuf[l & 1];
        a.xb_next = (l < L - 1 && h->use_tc) ? h->xbn[l & 1] : nullptr;
        a.xb_ld = h->ldn;
        a.xb_plane = (long long)h->max_T * h->max_B * h->ldn;
        a.xch = h->xch;
        a.status = h->status_dev;
        if (record(h, LSTM_K_RECUR, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        e = csr ? launch_recur_csr(a, bf16, shp.threads, shp.smem, st) : launch_recur_dense(a, bf16, shp.threads, shp.smem, st);
        ++h->last_launches;
        if (record(h, -1, st)) return fail(h, LSTM_ERR_CUDA, "event record failed");
        if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "recurrent launch failed (layer %d): %s", l, cudaGetErrorString(e));
        }
    }
    return LSTM_OK;
}

int lstm_input_projection(lstm_handle *h, const float *x, int T, int B, float *g, void *cuda_stream)
{
    if (!h) return LSTM_ERR_INVALID;
    if (T < 0 || B < 0 || T > h->max_T || B > h->max_B)
        return fail(h, LSTM_ERR_INVALID, "T=%d B=%d outside [0,%d] x [0,%d]", T, B, h->max_T, h->max_B);
    if (T == 0 || B == 0) return LSTM_OK;
    if (!x || !g) return fail(h, LSTM_ERR_INVALID, "x and g must not be NULL");
    if (h->inner) return fail(h, LSTM_ERR_UNSUPPORTED, "the projection on its own is not served on a compacted handle (create with LSTM_B200_COMPACT=0)");
    if (const int drc = check_device(h)) return drc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->last_stream = st;
    h->ev_used = 0;
    h->last_launches = 0;
    const int M = T * B, Hg = h->Hh ? h->Hh : h->H, N = h->D * 4 * Hg;
    int nsplit = 1;
    const int rc = run_projection(h, 0, x, x, M, N, &nsplit, st);
    if (rc != LSTM_OK) return rc;
    cudaError_t e = launch_proj_export(h->G, nsplit, (long long)M * N, g, M, h->D, Hg, st);
    ++h->last_launches;
    if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "export launch failed: %s", cudaGetErrorString(e));
    return LSTM_OK;
}

int lstm_status(lstm_handle *h)
{
    if (!h) return LSTM_ERR_INVALID;
    int v = 0;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    int *status_dev = h->inner ? h->inner->status_dev : h->status_dev;
    if (e == cudaSuccess) e = cudaMemcpy(&v, status_dev, sizeof v, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "status read failed: %s", cudaGetErrorString(e));
    if (v != 0) {
        cudaMemset(status_dev, 0, sizeof v);
        return fail(h, v, v == LSTM_ERR_TIMEOUT ? "a device-side wait gave up (timeout); outputs are undefined"
                          : v == LSTM_ERR_INTERNAL ? "an index check of the checked build failed inside a kernel; outputs are undefined"
                                                   : "device reported status %d", v);
    }
    return LSTM_OK;
}

int lstm_forward_host(lstm_handle *h, const float *x, int T, int B, const float *h0, const float *c0,
                      float *y, float *hT, float *cT, void *cuda_stream)
{
    if (!h) return LSTM_ERR_INVALID;
    if (T < 0 || B < 0 || T > h->max_T || B > h->max_B)
        return fail(h, LSTM_ERR_INVALID, "T=%d B=%d outside [0,%d] x [0,%d]", T, B, h->max_T, h->max_B);
    if (const int drc = check_device(h)) return drc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t Mmax = (size_t)h->max_T * h->max_B;
    const size_t smax = (size_t)h->L * h->D * h->max_B * h->H;
    if (!h->hx) {
        int rc = dev_alloc(h, &h->hx, Mmax * h->in_dim * 4, false, st, "host-variant x");
        if (!rc) rc = dev_alloc(h, &h->hy, Mmax * h->D * h->H * 4, false, st, "host-variant y");
        if (!rc) rc = dev_alloc(h, &h->hh0, smax * 4, false, st, "host-variant h0");
        if (!rc) rc = dev_alloc(h, &h->hc0, smax * 4, false, st, "host-variant c0");
        if (!rc) rc = dev_alloc(h, &h->hhT, smax * 4, false, st, "host-variant hT");
        if (!rc) rc = dev_alloc(h, &h->hcT, smax * 4, false, st, "host-variant cT");
        if (rc == LSTM_OK && cudaHostAlloc((void **)&h->status_pinned, sizeof(int), cudaHostAllocDefault) != cudaSuccess) {
            cudaGetLastError();
            rc = fail(h, LSTM_ERR_NOMEM, "pinned status word could not be allocated");
        }
        if (rc) return rc;
    }
    const size_t xn = (size_t)T * B * h->in_dim, yn = (size_t)T * B * h->D * h->H, sn = (size_t)h->L * h->D * B * h->H;
    cudaError_t e = cudaSuccess;
    if (xn && !x) return fail(h, LSTM_ERR_INVALID, "x must not be NULL");
    if (yn && !y) return fail(h, LSTM_ERR_INVALID, "y must not be NULL");
    if (xn) e = cudaMemcpyAsync(h->hx, x, xn * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && h0 && sn) e = cudaMemcpyAsync(h->hh0, h0, sn * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && c0 && sn) e = cudaMemcpyAsync(h->hc0, c0, sn * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(e));
    int rc = lstm_forward(h, h->hx, T, B, h0 ? h->hh0 : nullptr, c0 ? h->hc0 : nullptr, h->hy,
                          hT ? h->hhT : nullptr, cT ? h->hcT : nullptr, cuda_stream);
    if (rc) return rc;
    if (yn) e = cudaMemcpyAsync(y, h->hy, yn * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && hT && sn) e = cudaMemcpyAsync(hT, h->hhT, sn * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && cT && sn) e = cudaMemcpyAsync(cT, h->hcT, sn * 4, cudaMemcpyDeviceToHost, st);
    // the device status of this very call travels with the results: one synchronisation, no blocking copy
    int *status_dev = h->inner ? h->inner->status_dev : h->status_dev;
    *h->status_pinned = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->status_pinned, status_dev, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail(h, LSTM_ERR_CUDA, "device-to-host copy failed: %s", cudaGetErrorString(e));
    if (*h->status_pinned != 0) return lstm_status(h);         // reads, reports and clears the recorded status
    return LSTM_OK;
}

int lstm_destroy(lstm_handle *h)
{
    if (!h) return LSTM_OK;
    cudaDeviceSynchronize();
    if (h->inner) lstm_destroy(h->inner);
    free_all(h);
    delete h;
    return LSTM_OK;
}

int lstm_selftest_timeout(lstm_handle *h, int cta, long long spin_limit)
{
    if (!h) return LSTM_ERR_INVALID;
    if (h->inner) { const int rc = lstm_selftest_timeout(h->inner, cta, spin_limit); if (rc) h->err = h->inner->err; return rc; }
    if (cta >= h->ncta_dir * h->D) return fail(h, LSTM_ERR_INVALID, "cta %d outside the launch of %d CTAs", cta, h->ncta_dir * h->D);
    h->withhold_cta = cta < 0 ? -1 : cta;
    h->spin_limit = spin_limit > 0 ? spin_limit : h->spin_limit_default;
    return LSTM_OK;
}

int lstm_probe(lstm_handle *h, int parts_left_out)
{
    if (!h) return LSTM_ERR_INVALID;
    if (h->inner) { const int rc = lstm_probe(h->inner, parts_left_out); if (rc) h->err = h->inner->err; return rc; }
    if (parts_left_out < 0 || parts_left_out > 15) return fail(h, LSTM_ERR_INVALID, "probe mask %d outside 0..15", parts_left_out);
    if (parts_left_out && ((!h->use_mma && !h->use_csr_reg) || h->Hh))
        return fail(h, LSTM_ERR_UNSUPPORTED, "only the register-resident recurrent kernels (dense and sparse) of an LSTM handle have probe modes");
    h->probe = parts_left_out;
    return LSTM_OK;
}

int lstm_profile_enable(lstm_handle *h, int on)
{
    if (!h) return LSTM_ERR_INVALID;
    if (h->inner) return lstm_profile_enable(h->inner, on);
    h->prof = on != 0;
    h->ev_used = 0;
    return LSTM_OK;
}

int lstm_profile_read(lstm_handle *h, int *launches, float *ms)
{
    if (!h || !launches || !ms) return LSTM_ERR_INVALID;
    if (h->inner) { const int rc = lstm_profile_read(h->inner, launches, ms); if (rc) h->err = h->inner->err; return rc; }
    for (int k = 0; k < LSTM_K_COUNT; ++k) { launches[k] = 0; ms[k] = 0.0f; }
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess)
        return fail(h, LSTM_ERR_CUDA, "synchronise failed: %s", cudaGetErrorString(cudaGetLastError()));
    for (int i = 0; i + 1 < h->ev_used; i += 2) {
        const int k = h->ev_kind[i];
        float t = 0.0f;
        if (k < 0 || k >= LSTM_K_COUNT) continue;
        if (cudaEventElapsedTime(&t, h->ev[i], h->ev[i + 1]) != cudaSuccess)
            return fail(h, LSTM_ERR_CUDA, "event timing failed: %s", cudaGetErrorString(cudaGetLastError()));
        launches[k] += 1;
        ms[k] += t;
    }
    return LSTM_OK;
}

int lstm_info(const lstm_handle *h, int64_t *out, int n)
{
    if (!h || !out || n < 0) return 0;
    if (h->inner) {
        const int cnt = lstm_info(h->inner, out, n);
        if (n > 8) out[8] = h->last_launches > 0 ? h->last_launches : out[8] + 1;
        if (n > 16) out[16] = h->Hc;
        if (n > 17) out[17] = h->n_removed;
        return cnt;
    }
    RecurShape shp = recur_shape(h, h->max_B, 0);
    if (h->Hh) shp.smem = hlstm_mma_smem_bytes(h->mma_mt, h->mma_nkr, h->mma_nw, h->mma_nks, h->hl_nkw2, h->upc, h->max_B);
    const size_t wsize = h->dtype == LSTM_BF16W_F32S ? 2 : 4;
    int64_t rows_res = 0, rows_str = 0;
    if (h->use_mma) {
        rows_res = 4 * h->upc;
    } else if (h->exec_mode == LSTM_DENSE) {
        const size_t unit_bytes = (size_t)4 * h->Hp8 * wsize;
        const int ures = (int)std::min<size_t>(h->upc, shp.w_smem_bytes / unit_bytes);
        rows_res = 4 * ures; rows_str = 4 * (h->upc - ures);
    }
    const Layer &l0 = h->layers[0];
    const int launches = h->last_launches > 0 ? h->last_launches : h->L * 2 + (h->use_tc ? 1 : 0);
    int ik = 0, is = 0;
    const int tcb_at_max = (h->use_tcb && !h->Hh && h->max_B > 4 && h->max_B <= kTcMaxBatch &&
                            recur_tc_plan(h->tcb_RA, h->tcb_nkb, round_up(2 * h->max_B, 16), h->upc, h->max_B, (size_t)h->smem_optin - kTcStaticSmem,
                                          h->tcb_pair ? 1 : 0, &ik, &is)) ? (h->tcb_pair ? 2 : 1) : 0;
    if (h->use_csr_reg) shp.smem = recur_csr_reg_smem_bytes(h->csr_nw, h->csr_kspan, h->csr_mt, h->upc, h->max_B);
    const int64_t vals[19] = {h->sm_count, h->ncta_dir, h->use_mma ? h->mma_nw * 32 : h->use_csr_reg ? h->csr_nw * 32 : h->threads, (int64_t)shp.smem,
                              rows_res, rows_str, (l0.plan_M >= 0) ? l0.plan.nsplit : 1, h->use_tc ? 1 : 0, launches,
                              h->use_mma ? 1 : 0, h->use_mma ? h->mma_nkr : 0, h->use_mma ? h->mma_nks : 0, tcb_at_max,
                              h->use_csr_reg ? 1 : 0, h->use_csr_reg ? h->csr_slots : 0, h->use_csr_reg ? h->csr_conflicts : 0, 0, 0, h->use_wave ? 1 : 0};
    for (int i = 0; i < n && i < 19; ++i) out[i] = vals[i];
    return 19;
}

}  // extern "C"
