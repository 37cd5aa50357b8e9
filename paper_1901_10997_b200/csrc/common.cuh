// Shared declarations of the lstm_b200 library: kernel argument blocks and launch entry points.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace lstm {

// device status word values (mirrors the LSTM_* return codes of the C header)
constexpr int kStatusOk = 0;
constexpr int kStatusTimeout = 5;

// ---------------------------------------------------------------------------------------------------
// Recurrent kernel (dense and CSR).  One cooperative launch per layer covers both directions: CTAs
// [0, ncta_dir) run direction 0, CTAs [ncta_dir, 2*ncta_dir) direction 1.  Hidden units are split
// evenly over a direction's CTAs; CTA c owns units [u0(c), u0(c) + n(c)).
// ---------------------------------------------------------------------------------------------------
struct RecurArgs {
    int dir0, ndirs;            // directions this launch runs: dir0 .. dir0 + ndirs - 1 (ndirs = 0 means all D)
    int H;              // hidden width
    int Hp8;            // dense: row length of the packed recurrent matrix (H rounded up to 8)
    int Hs;             // length of one staged h row in shared memory (H rounded up to 256)
    int B, T, D;
    int ncta_dir;       // CTAs per direction
    int nsplit;         // partial planes of the projection output to add up
    int BT;             // batch rows processed per chunk (1, 2, 4 or 8)
    int w_smem_bytes;   // shared-memory bytes set aside for resident weights
    int stage_all;      // 1: all B rows of h are staged at once (one polling phase per step), chunks of BT rows share them
    unsigned stamp_base;        // exchange words of step s carry stamp_base + s + 1
    long long spin_limit;       // clock64 ticks a wait may last before the kernel gives up
    int withhold_cta;           // failure-path self-test: this CTA never publishes its h values (-1: none)
    // dense: [H][4][Hp8] (unit-major, gates i,f,g,o); element type = weight type
    const void *wh[2];
    // CSR: per direction, rows in the same unit-major order; entry_ptr[4H+1] counts entries padded
    // per row to a multiple of 4; entries are {col<<16 | bf16} words (bf16) or {val, col} pairs (fp32)
    const int *csr_ptr[2];
    const void *csr_ent[2];
    const float *G;             // [nsplit][T*B][D][H][4] projection output incl. bias
    long long g_split_stride;   // elements between partial planes
    const float *h0, *c0;       // [D][B][H] of this layer or nullptr
    float *hT, *cT;             // [D][B][H] of this layer or nullptr
    float *y;                   // [T][B][D*H]
    __nv_bfloat16 *xb_next;     // y as two bf16 terms (hi plane, then lo plane) for the next layer's
    long long xb_plane;         //   tensor-core projection, or nullptr; elements between the planes
    int xb_ld;                  // row stride in elements
    unsigned long long *xch;    // [D][2][B][H] exchange words {stamp:32 | h bits:32}
    int *status;                // device status word
};

cudaError_t launch_recur_dense(const RecurArgs &a, bool bf16_weights, int threads, size_t smem,
                               cudaStream_t st);
cudaError_t launch_recur_csr(const RecurArgs &a, bool bf16_weights, int threads, size_t smem,
                             cudaStream_t st);
cudaError_t recur_dense_prepare(int max_smem);   // raises the dynamic shared-memory limit once
cudaError_t recur_csr_prepare(int max_smem);

// ---------------------------------------------------------------------------------------------------
// Register-resident recurrent kernel (bf16 weights, dense).  Same CTA/unit partition and exchange
// buffer as above.  The slice of a CTA is cut into 16 x 16 tiles: MT row tiles (4 gate rows per unit,
// zero-padded) by NW * nkw column tiles; warp w owns column tiles [w * nkw, (w + 1) * nkw) of every row
// tile, the first NKR of them in registers, the remaining nkw_smem in shared memory.
// ---------------------------------------------------------------------------------------------------
struct RecurMmaArgs {
    int dir0, ndirs;            // directions this launch runs: dir0 .. dir0 + ndirs - 1 (ndirs = 0 means all D)
    int H, B, T, D;
    int ncta_dir;
    int nsplit;
    int nkw_smem;               // trailing column tiles of every warp kept in shared memory
    int staged;                 // 1: passes over several batch rows land their exchange words in shared memory
    unsigned stamp_base;
    long long spin_limit;
    int withhold_cta;           // failure-path self-test: this CTA never publishes its h values (-1: none)
    int probe;                  // measurement only (kProbe* bits): parts of a step left out, outputs undefined
    // fused input projection (one sequence of at most kFuseMaxT steps): the CTA computes its rows of G itself
    int fuse;                   // 1: G is not read; X, xfrag, bias, in_l, nkw_x describe the projection
    int in_l, nkw_x;            // input width; column tiles of Wx per column range (NW / 2 ranges, two warps each)
    int gs_off;                 // byte offset of the finished rows of G in dynamic shared memory
    const float *X;             // [T][in_l] this layer's input (fp32)
    const uint4 *xfrag[2];      // Wx per direction in the fragment layout below with NW / 2 ranges of nkw_x tiles
    const float *bias;          // [D][H][4]
    // per direction [cta][warp][column tile][row tile][lane] 16-byte operand-A fragments:
    // lane (g = lane / 4, p = lane % 4) holds rows g and g + 8, columns 2p, 2p+1 and 2p+8, 2p+9
    const uint4 *wfrag[2];
    const float *G;
    long long g_split_stride;
    const float *h0, *c0;
    float *hT, *cT;
    float *y;
    __nv_bfloat16 *xb_next;
    long long xb_plane;
    int xb_ld;
    unsigned long long *xch;
    int *status;
};
// probe bits of the register-resident kernels: what a step leaves out when its cost is being measured
constexpr int kProbeNoProducts = 1;   // no tensor instructions (partial sums are written as zeros)
constexpr int kProbeNoGates = 2;      // no reduction, gate functions or output stores: the unit's word is published as it is
constexpr int kProbeNoExchange = 4;   // no wait for the other CTAs' words
constexpr int kMmaTileCap16 = 18;   // MT * NKR limit with 16 warps (128 registers per thread, no spills)
constexpr int kMmaTileCap8 = 40;    // ... with 8 warps
bool recur_mma_shape_ok(int mt, int nkr, int nw);
size_t recur_mma_smem_bytes(int mt, int nkr, int nw, int nkw_smem, int upc, int B, bool staged, bool fused = false);
size_t recur_mma_fuse_gs_offset(int mt, int nkr, int nw, int nkw_smem, int upc);
constexpr int kFuseMaxT = 40;        // longest sequence whose projection the recurrent kernel computes in its prologue
cudaError_t recur_mma_prepare(int mt, int nkr, int nw, int max_smem);
cudaError_t launch_recur_mma(const RecurMmaArgs &a, int mt, int nkr, int nw, size_t smem, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// Layer-wavefront recurrent kernel (unidirectional stacks of 2 to 4 layers, bf16 dense, up to four sequences).
// CTAs [l * ncta_layer, (l + 1) * ncta_layer) run layer l.  Layer 0's matrix is Wh_0 [4H x H]; layer l >= 1's
// is [Wx_l | Wh_l] [4H x 2H] acting on [h^{l-1}_t ; h^l_{t-1}].  Fragment layout as in RecurMmaArgs with
// nkw[l] column tiles per warp (the first NKR in registers).
// ---------------------------------------------------------------------------------------------------
constexpr int kMaxWaveLayers = 4;
constexpr int kWaveTileCap = 16;     // MT * NKR limit (128 registers per thread at 16 warps, no spills)
struct RecurWaveArgs {
    int L, H, B, T;
    int ncta_layer;
    int nsplit;                 // partial planes of layer 0's projection output
    int nkw[kMaxWaveLayers];    // column tiles per warp of each layer's CTAs (>= the register tiles)
    int nkw_max;
    unsigned stamp_base;        // the word of (layer, step s) carries stamp_base + s + 1
    long long spin_limit;
    int withhold_cta;
    const uint4 *wfrag[kMaxWaveLayers];
    const float *bias[kMaxWaveLayers];   // [H][4] (unit-major) bias of layers >= 1; layer 0's is in G
    const float *G;             // [nsplit][T*B][H][4] layer 0's projection output incl. bias
    long long g_split_stride;
    const float *h0, *c0;       // [L][B][H] or nullptr
    float *hT, *cT;             // [L][B][H] or nullptr
    float *y;                   // [T][B][H]: the top layer's h
    unsigned long long *xch;    // [L][T][B][H] exchange words, one slot per (layer, timestep)
    int *status;
};
bool recur_wave_shape_ok(int mt, int nkr);
size_t recur_wave_smem_bytes(int mt, int nkr, int nkw_max, int upc, int B);
cudaError_t recur_wave_prepare(int mt, int nkr, int max_smem);
cudaError_t launch_recur_wave(const RecurWaveArgs &a, int mt, int nkr, size_t smem, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// Register-resident sparse recurrent kernel (bf16 weights, CSR execution).  Same CTA/unit partition,
// exchange buffer and finishing role as the dense register-resident kernel.  Warp w of a CTA owns the
// columns [w * kspan, (w + 1) * kspan) of h; inside the warp every lane owns up to two of the CTA's 4 * units
// gate rows and keeps the surviving weights of those rows in that column range in registers for the whole
// sequence, one 32-bit word each: {bf16 value : 16 | second-row flag : 1 | column inside the range : 15}.
// A launch is compiled for E entry slots per lane; shorter lists are padded with zero words.
// ---------------------------------------------------------------------------------------------------
struct RecurCsrArgs {
    int dir0, ndirs;            // directions this launch runs: dir0 .. dir0 + ndirs - 1 (ndirs = 0 means all D)
    int H, B, T, D;
    int ncta_dir;
    int nsplit;
    int kspan;                  // columns of h per warp (multiple of 32)
    int hs_stride;              // floats of a warp's staging block: power of two >= rows per pass * kspan (set by the launcher)
    int mt;                     // 16-row tiles that cover 4 * units per CTA (sets the pitch of the partial sums)
    unsigned stamp_base;
    long long spin_limit;
    int withhold_cta;
    int probe;                  // kProbe* bits, single-sequence calls only
    const unsigned *ent[2];     // per direction [cta][warp][E][32 lanes] entry words
    const unsigned *rows[2];    // per direction [cta][warp][32 lanes]: local rows of the lane's two lists
                                //   (byte 0: first, byte 1: second; 0xff: none)
    const float *G;
    long long g_split_stride;
    const float *h0, *c0;
    float *hT, *cT;
    float *y;
    __nv_bfloat16 *xb_next;
    long long xb_plane;
    int xb_ld;
    unsigned long long *xch;
    int *status;
    // projection fused into the prologue (single sequence, T <= kFuseMaxT): Wx as operand-A fragments of a dense
    // copy (zeros included), layout as in RecurMmaArgs with NW / 2 column ranges
    int fuse, in_l, nkw_x, gs_off;
    const float *X, *bias;
    const uint4 *xfrag[2];
};
size_t recur_csr_reg_fuse_gs_offset(int nw, int kspan, int mt, int upc);
size_t recur_csr_reg_fuse_smem_bytes(int nw, int kspan, int mt, int upc);
constexpr int kCsrRegMaxSlots16 = 64;    // entry slots per lane the kernel is built for with 16 warps ...
constexpr int kCsrRegMaxSlots8 = 128;    // ... and with 8 warps (255 registers per thread)
int recur_csr_reg_slots(int needed, int nw);     // smallest built slot count >= needed, or 0 when none is
size_t recur_csr_reg_smem_bytes(int nw, int kspan, int mt, int upc, int B);
cudaError_t recur_csr_reg_prepare(int slots, int nw, int max_smem);
cudaError_t launch_recur_csr_reg(const RecurCsrArgs &a, int slots, int nw, size_t smem, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// Batched recurrent kernel on tcgen05 (bf16 weights, dense, more than four batch rows).  The CTA's slice of
// Wh sits in shared memory as K-major 128-byte-swizzled tiles of RA rows (4 * units per CTA rounded up to 8)
// per 64 columns; h travels through global memory as bf16 planes [D][2 parities][64 rows][ldh] (row 2b = hi,
// 2b+1 = lo part of batch row b) and one stamp per producer CTA.
// ---------------------------------------------------------------------------------------------------
constexpr int kTcMaxBatch = 64;       // sequences per call the batched tensor-core recurrence serves
constexpr int kTcStaticSmem = 1024;   // bytes kept free for the kernel's static shared memory (barriers, flags: under 600)
constexpr int kTcPlaneRows = 128;     // rows of one parity of the h planes: hi and lo row of every sequence
struct RecurTcArgs {
    int dir0, ndirs;            // directions this launch runs: dir0 .. dir0 + ndirs - 1 (ndirs = 0 means all D)
    int H, B, T, D;
    int ncta_dir;
    int nsplit;
    int RA, nkb;                // rows of a weight tile; 64-column K blocks
    int N;                      // MMA N: 2 * B rounded up to 16
    int stages;                 // depth of the operand ring
    int kbs;                    // K blocks per ring stage
    int pair;                   // 1: clusters of two CTAs split K (launched with cluster dimension 2)
    int nissue;                 // threads issuing tensor instructions, each with its own accumulator: 1 to 3, <= K blocks of any CTA
    int tmem_cols;              // power of two >= max(32, nissue * N)
    int ldh;                    // row stride of the planes (elements, multiple of 8)
    unsigned stamp_base;
    long long spin_limit;
    int withhold_cta;
    const float *G;
    long long g_split_stride;
    const float *h0, *c0;
    float *hT, *cT;
    float *y;
    __nv_bfloat16 *xb_next;
    long long xb_plane;
    int xb_ld;
    __nv_bfloat16 *hbuf;
    unsigned *flags;            // [D][ncta_dir]
    int *status;
};
size_t recur_tc_smem_bytes(int RA, int nkb, int N, int stages, int kbs, int upc, int B, int pair);
bool recur_tc_plan(int RA, int nkb, int N, int upc, int B, size_t max_smem, int pair, int *kbs_out, int *stages_out);
bool recur_tc_pair_supported(int grid, size_t smem);
bool recur_tc_encode_weights(void *map128, const void *w, long long rows, int ld, int RA);
bool recur_tc_encode_planes(void *map128, const void *hbuf, int D, int H, int ldh, int B);
cudaError_t recur_tc_prepare(int max_smem);
cudaError_t launch_recur_tc(const void *tmap_w, const void *tmap_h, const RecurTcArgs &a, size_t smem, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// H-LSTM recurrent kernel (one ReLU hidden layer of width Hh inside each gate; bf16 weights, dense).
// Pass 1 works on the four Uh_q [Hh x H] (hidden units split over the CTAs, fragments in registers and,
// beyond nkr tiles per warp, in shared memory), pass 2 on the four W_q [H x Hh] (cell units split over the
// CTAs, fragments in shared memory).  Fragment layout as in RecurMmaArgs.
// ---------------------------------------------------------------------------------------------------
struct HlstmArgs {
    int dir0, ndirs;            // directions this launch runs: dir0 .. dir0 + ndirs - 1 (ndirs = 0 means all D)
    int H, Hh, B, T, D;
    int ncta_dir;
    int nsplit;
    int nks1;                   // pass 1: column tiles per warp in shared memory (after the register tiles)
    int nkw2;                   // pass 2: column tiles per warp (all in shared memory)
    unsigned stamp_base;
    long long spin_limit;
    int withhold_cta;
    const uint4 *frag1[2];      // Uh: local row = 4 * hidden unit + gate
    const uint4 *frag2[2];      // W:  local row = 4 * cell unit + gate
    const float *G;             // [nsplit][T*B][D][Hh][4] input half of the hidden layers incl. their bias
    long long g_split_stride;
    const float *bias_out;      // [D][H][4] bias of the gate pre-activations
    const float *h0, *c0;
    float *hT, *cT;
    float *y;
    __nv_bfloat16 *xb_next;
    long long xb_plane;
    int xb_ld;
    unsigned long long *xch;    // [D][2][B][H] h words
    unsigned long long *rxch;   // [D][2][B][4][Hh] hidden-layer words
    int *status;
};
size_t hlstm_mma_smem_bytes(int mt, int nkr, int nw, int nks1, int nkw2, int upc, int B);
cudaError_t hlstm_mma_prepare(int mt, int nkr, int nw, int max_smem);
cudaError_t launch_hlstm_mma(const HlstmArgs &a, int mt, int nkr, int nw, size_t smem, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// Row/column-pruned stacks: moving states and outputs between the full width H and the compact width Hc of the
// surviving units, and the closed-form recurrence of the removed ones.
// ---------------------------------------------------------------------------------------------------
struct CompactArgs {
    int L, D, H, Hc, T, B;
    const int *cmap;            // [L*D][Hc]: unit of the full model behind compact unit jc
    int n_removed;
    const int *rem_idx;         // [n_removed][2]: {layer * D + direction, unit}
    const float *rem_bias;      // [n_removed][4]: b_i, b_f, b_g, b_o of the removed unit
    const float *h0, *c0;       // caller's [L*D][B][H] or nullptr
    float *h0c, *c0c;           // compact [L*D][B][Hc]
    const float *yc;            // compact [T][B][D*Hc]
    const float *hTc, *cTc;     // compact [L*D][B][Hc]
    float *y;                   // caller's [T][B][D*H]
    float *hT, *cT;             // caller's [L*D][B][H] or nullptr
};
cudaError_t launch_compact_gather(const CompactArgs &a, cudaStream_t st);
cudaError_t launch_compact_scatter(const CompactArgs &a, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------
// Input staging and projection
// ---------------------------------------------------------------------------------------------------
// x fp32 [M][K] -> two bf16 planes [M][ld]: hi = bf16(x), lo = bf16(x - hi) at xb + plane
// (columns K..ld-1 are written as zero)
cudaError_t launch_stage_bf16(const float *x, __nv_bfloat16 *xb, long long plane, long long M, int K, int ld,
                              cudaStream_t st);

// G[m][n] = sum_k X[m][k] * W[n][k] + bias[n];  X fp32 [M][K], W [N][ldw] fp32 or bf16, G fp32 [M][N]
cudaError_t launch_proj_simt(const float *X, const void *W, bool bf16_weights, int ldw,
                             const float *bias, float *G, int M, int N, int K, cudaStream_t st);

// G[m][n] = sum_e val[e] * X[m][col[e]] + bias[n] over CSR row n (entries {val,col} pairs)
struct CsrEntry { float val; int col; };
cudaError_t proj_csr_prepare(int max_smem);   // raises the dynamic shared-memory limit once
cudaError_t launch_proj_csr(const float *X, const int *rowptr, const CsrEntry *ent,
                            const float *bias, float *G, int M, int N, int K, bool f64_acc, cudaStream_t st);

// out[m][d][q][j] = sum over split planes of G[split][m][d][j][q]: the projection in the public layout
// (gate blocks i,f,g,o of Hg rows per direction) from the internal unit-major one
cudaError_t launch_proj_export(const float *G, int nsplit, long long split_stride, float *out, long long M, int D, int Hg,
                               cudaStream_t st);

// Tensor-core projection (tcgen05 + TMEM + TMA).  A = packed weights [N][ldk] bf16 (K-major),
// activations [M][ldk] as two bf16 planes (hi, lo); writes G[split][M][N] fp32 (+bias on split 0).
struct ProjTcPlan {
    alignas(64) unsigned char tmap_w[128];
    alignas(64) unsigned char tmap_x[128];
    alignas(64) unsigned char tmap_xlo[128];
    int M, N, K, ldk;
    int n_tile;        // MMA N extent (activation rows per tile), multiple of 16, <= 256
    int nsplit;        // split-K factor
    int kblocks;       // ceil(K / 64)
    int sm_count;      // CTAs of the persistent kernel that serves shapes with several activation tiles
};
int  proj_tc_plan(ProjTcPlan *p, const __nv_bfloat16 *W, const __nv_bfloat16 *X, const __nv_bfloat16 *Xlo,
                  int M, int N, int K, int ldk, int sm_count, char *err, int errlen);
cudaError_t launch_proj_tc(const ProjTcPlan &p, const float *bias, float *G, int *status,
                           cudaStream_t st);
cudaError_t proj_tc_prepare();

}  // namespace lstm
