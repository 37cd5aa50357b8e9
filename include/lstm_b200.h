/*
 * lstm_b200 -- stacked (optionally bidirectional) LSTM inference forward pass on one sm_100a GPU.
 *
 * C ABI: plain pointers and sizes only.  Every function returns one of the LSTM_* codes below (except
 * lstm_last_error); on failure lstm_last_error(handle) -- or lstm_last_error(NULL) for a failed
 * lstm_create -- returns a human-readable reason.  No function falls back to the CPU: without a usable
 * CUDA device every call fails with LSTM_ERR_CUDA.
 *
 * What is computed (paper, Section 4, the cell-equation block, with zero hidden layers inside each
 * gate, i.e. the conventional LSTM the paper takes as its baseline in Sections 5.1 and 5.2).  For
 * layer l, direction d, timestep t in processing order (forward 0..T-1; reverse T-1..0), batch row b,
 * hidden unit j, with W = [Wx | Wh] acting on the concatenation [x_t, h_{t-1}]:
 *
 *     z_q[j] = b_q[j] + sum_k Wx_q[j,k] X_l[t,b,k] + sum_k Wh_q[j,k] h_prev[b,k]     q in {i,f,g,o}
 *     i = sigmoid(z_i)  f = sigmoid(z_f)  g = tanh(z_g)  o = sigmoid(z_o)
 *     c = f * c_prev + i * g             h = o * tanh(c)
 *
 * X_0 = x; X_l for l > 0 is the previous layer's output [T,B,D*H] (forward half first, then reverse).
 * Pruned weights follow the mask-based scheme of Section 4: the effective matrix is W (x) Msk.
 *
 * Layout conventions
 *   - Gate rows are packed in four blocks of H rows in the order i, f, g, o: row q*H + j.
 *   - All activations are fp32, contiguous, time-major: x [T,B,in_dim], y [T,B,D*H].
 *   - State tensors are [L*D, B, H]; entry l*D + d (d = 1 is the reverse direction).  The reverse
 *     direction starts from h0/c0[l*D+1] at t = T-1 and its final state is the one after t = 0.
 *   - A handle is bound to the device that was current in lstm_create; calls on one handle must not
 *     overlap (one handle is not thread-safe); different handles are independent.
 */
#ifndef LSTM_B200_H
#define LSTM_B200_H

#include <stdint.h>

#if defined(__GNUC__)
#define LSTM_API __attribute__((visibility("default")))
#else
#define LSTM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lstm_handle lstm_handle;      /* opaque, library-owned */

/* storage / arithmetic type */
enum {
    LSTM_F32       = 0,   /* fp32 weights, activations, state and outputs; dot products and gate
                             functions are evaluated in fp64 (fp32 sums miss the 1e-4 bound near zero)  */
    LSTM_BF16W_F32S = 1   /* weights rounded to bf16 (nearest-even) at create time; the input
                             projection feeds the tensor cores with each activation as two bf16
                             terms (hi + lo, about 16 mantissa bits); state, accumulation, gates and
                             outputs are fp32                                                           */
};

/* return codes */
enum {
    LSTM_OK = 0,
    LSTM_ERR_INVALID = 1,      /* bad argument (NULL, shape, T > max_T, malformed CSR ...); nothing launched */
    LSTM_ERR_UNSUPPORTED = 2,  /* valid request the library cannot serve (e.g. hidden >= 65536)            */
    LSTM_ERR_CUDA = 3,         /* a CUDA call failed (no device, launch refused ...)                        */
    LSTM_ERR_NOMEM = 4,        /* host or device allocation failed                                           */
    LSTM_ERR_TIMEOUT = 5,      /* a device-side wait of the recurrent kernel gave up; outputs undefined     */
    LSTM_ERR_INTERNAL = 6      /* checked build only (liblstm_b200_checked.so, compiled with -DLSTM_B200_CHECKED):
                                  an index or shared-memory carve-up check inside a kernel failed; the access
                                  was skipped, nothing trapped; outputs undefined                            */
};

/* how the recurrent and input matrices are executed */
enum {
    LSTM_DENSE = 0,   /* dense kernels; a mask, if given, is applied as explicit zeros                 */
    LSTM_CSR   = 1    /* sparse kernels over the surviving entries only (from masks or caller CSR)      */
};

/*
 * Weights of one (layer, direction); array index = layer*D + direction.  All pointers may be host or
 * device pointers (the library finds out which) and are only read during lstm_create; the caller may
 * free them afterwards.
 *   dense form:  wx [4H, in_l], wh [4H, H] row-major fp32 (in_l = in_dim for layer 0, D*H after);
 *                optional masks of the same shapes, uint8, 1 = keep (the paper's Msk), NULL = keep all.
 *   CSR form:    used for a matrix when its rowptr is non-NULL (then the dense pointer and mask of
 *                that matrix are ignored): rowptr int32[4H+1] starting at 0, col int32[nnz] strictly
 *                increasing inside each row and within range, val fp32[nnz].
 *   b:           [4H] single bias per gate (a two-bias convention passes the sum); NULL = zeros.
 */
typedef struct {
    const float   *wx;
    const float   *wh;
    const float   *b;
    const uint8_t *mask_x;
    const uint8_t *mask_h;
    const int32_t *wx_rowptr; const int32_t *wx_col; const float *wx_val;
    const int32_t *wh_rowptr; const int32_t *wh_col; const float *wh_val;
} lstm_weights;

/*
 * Create-time packing (Section 4: W <- W (x) Msk once training has finished; here: once, at create).
 * Copies, masks, rounds (bf16 mode) and re-tiles all weights into library-owned device memory, and
 * allocates the workspace for sequences up to max_T steps and max_B batch rows.
 *   layers >= 1, in_dim >= 1, 1 <= hidden < 65536, bidir in {0,1}, dtype LSTM_F32 | LSTM_BF16W_F32S,
 *   w[layers*(1+bidir)], exec_mode LSTM_DENSE | LSTM_CSR, 1 <= max_T, 1 <= max_B,
 *   cuda_stream: a cudaStream_t (NULL = default stream) used for the uploads.
 * Synchronises the stream before returning.  On failure *out is NULL.
 * Environment switches read at create time (for measurements and tests; unset = the library chooses):
 *   LSTM_B200_RECUR = simt  shared-memory recurrent kernel instead of the register-resident one (bf16 dense or CSR)
 *                   = mma   no batched tensor-core recurrence (batches above four run as passes of four)
 *                   = tc1   batched tensor-core recurrence without cluster pairs
 *   LSTM_B200_FUSE  = 0     never compute the input projection inside the recurrent kernel (single sequences of up
 *                           to 40 steps on the register-resident kernel do so by default)
 *   LSTM_B200_WAVE  = 0     one launch per layer even where the layer-wavefront kernel would serve the stack
 *   LSTM_B200_PROJ  = simt  CUDA-core input projection instead of the tensor-core one
 *                   = csr   CSR handles walk the lists of Wx in the projection too (by default bf16 CSR handles keep a
 *                           dense copy of Wx and project on the tensor cores; the recurrence stays sparse)
 *   LSTM_B200_PROJ_TILE = 128  the 128-row-tile projection kernel (two CTAs per SM) also where the persistent
 *                           256-row-tile kernel would run (several activation tiles)
 *   LSTM_B200_PROJ_SMEM_KB = 48..200  shared-memory budget of the 128-row-tile projection kernel (ring depth)
 *   LSTM_B200_CTAS  = <n>   at most n CTAs per direction in the recurrent kernels (measurement)
 *   LSTM_B200_TC_ISSUE = 1|2  fewer issuing threads (and accumulators) in the batched tensor-core recurrence than the
 *                           three it uses where the K extent allows
 *   LSTM_B200_COMPACT = 0   keep row/column-pruned units as explicit zeros, = 1 always run on the surviving units
 *                           (unset: handles with max_B >= 5 compact, smaller ones keep the zeros; see below)
 * Row/column-pruned stacks (Section 4.2, Algorithm 1: whole rows and columns of the gate matrices are zero).
 * lstm_create (for max_B >= 5, or when LSTM_B200_COMPACT=1) looks for hidden units that read nothing and are read by nobody: all four gate rows zero in Wx and
 * Wh, the unit's column of Wh zero and, below the last layer, its column of every next-layer Wx zero.  If every
 * (layer, direction) has such units, the forward pass runs on the surviving units only, at the compact width
 * Hc = the largest number of survivors of any matrix (what the paper's pruning buys on a GPU: a smaller dense
 * model); the removed units' outputs and final states follow from their biases and c0 in closed form
 * (constant gates) and are written beside the survivors', so y, hT and cT keep the full width and the result
 * equals the dense-with-zeros one.  Such a handle costs one small extra kernel per call (two when h0 or c0 is
 * given) and does not serve lstm_input_projection.  Handles for up to four sequences keep the zeros by default:
 * their step is bound by the exchange latency, not by the width, and the extra kernel would cost more than the
 * narrower model saves.
 *   LSTM_B200_SPIN_LIMIT = <clock ticks>  bound of every device-side wait (default about two seconds)
 */
LSTM_API int lstm_create(lstm_handle **out, int layers, int in_dim, int hidden, int bidir, int dtype,
                const lstm_weights *w, int exec_mode, int max_T, int max_B, void *cuda_stream);

/*
 * H-LSTM cell (Section 4 with one hidden layer H inside each gate: a linear map followed by ReLU).  For
 * gate q in {i,f,g,o}, hidden width Hh = gate_hidden:
 *     r_q = relu(a_q + Ux_q x_t + Uh_q h_{t-1})        z_q = b_q + W_q r_q
 * followed by the same gate functions and c/h update as above.  Weights of one (layer, direction), all
 * row-major fp32, host or device pointers, read only during the call:
 *   ux [4Hh, in_l], uh [4Hh, H]: rows q*Hh + m;  a [4Hh] or NULL;  w [4H, Hh]: row q*H + j multiplies r_q;
 *   b [4H] or NULL.  Pruned weights: explicit zeros in ux, uh, w, or the keep-masks below.
 * hlstm_create returns a handle that lstm_forward, lstm_forward_host, lstm_status, lstm_destroy and the
 * other calls accept like an LSTM handle.  Only LSTM_BF16W_F32S storage is served; sizes whose per-CTA
 * slices of Uh and W do not fit registers + shared memory (roughly hidden, gate_hidden > 1700) return
 * LSTM_ERR_UNSUPPORTED.
 */
typedef struct {
    const float *ux;
    const float *uh;
    const float *a;
    const float *w;
    const float *b;
    /* optional keep-masks (Section 4.2: W (x) Msk), one byte per weight, non-zero = kept, same shapes as ux, uh
     * and w; NULL keeps every weight.  A masked weight is multiplied as an explicit zero. */
    const unsigned char *mask_ux;
    const unsigned char *mask_uh;
    const unsigned char *mask_w;
} hlstm_weights;

LSTM_API int hlstm_create(lstm_handle **out, int layers, int in_dim, int hidden, int gate_hidden, int bidir, int dtype,
                 const hlstm_weights *w, int max_T, int max_B, void *cuda_stream);

/*
 * Forward pass over a whole sequence batch; all pointers are DEVICE pointers owned by the caller.
 *   x  [T,B,in_dim]      h0, c0 [L*D,B,H] or NULL (zeros)
 *   y  [T,B,D*H]         hT, cT [L*D,B,H] or NULL (not wanted)
 * 0 <= T <= max_T, 0 <= B <= max_B (T = 0 or B = 0: nothing is launched; hT,cT receive h0,c0).
 * Work is enqueued on cuda_stream and the call returns without synchronising; a device-side timeout
 * of this call is reported by lstm_status on the handle.
 * Steps, in order, per layer: input staging (bf16 mode), input projection for all timesteps at once
 * (the x_t half of W [x_t, h_{t-1}] + b), then the serial recurrence with the gate nonlinearities and
 * the c/h update fused into one persistent kernel.
 */
LSTM_API int lstm_forward(lstm_handle *h, const float *x, int T, int B, const float *h0, const float *c0,
                 float *y, float *hT, float *cT, void *cuda_stream);

/*
 * Same computation with HOST buffers (pinned or pageable): copies x (and h0, c0 if given) to
 * handle-owned device staging buffers, runs lstm_forward, copies y (and hT, cT if wanted) back, and
 * synchronises cuda_stream before returning, so the device status of this very call is returned.
 */
LSTM_API int lstm_forward_host(lstm_handle *h, const float *x, int T, int B, const float *h0, const float *c0,
                      float *y, float *hT, float *cT, void *cuda_stream);

/*
 * The input projection of the first layer on its own (the x_t half of W [x_t, h_{t-1}] + b for all
 * timesteps at once; the dense-versus-sparse matrix product the paper times in Section 3, Figures 1, 2):
 *     g[t,b,d,q*Hg + j] = bias_q[j] + sum_k Wx_{d,q}[j,k] x[t,b,k]
 * x [T,B,in_dim] and g [T,B,D,4*Hg] are DEVICE pointers (Hg = hidden, or gate_hidden for an H-LSTM handle
 * where the rows are those of Ux and the bias is a); gate blocks i,f,g,o.  Runs the same staging and
 * projection kernels as lstm_forward (tensor-core, CUDA-core or CSR according to the handle) plus a small
 * re-layout kernel; enqueued on cuda_stream without synchronising.  0 <= T <= max_T, 0 <= B <= max_B.
 */
LSTM_API int lstm_input_projection(lstm_handle *h, const float *x, int T, int B, float *g, void *cuda_stream);

/* Synchronises the stream last used with the handle and returns LSTM_OK or the recorded device
 * status (LSTM_ERR_TIMEOUT ...); the recorded status is cleared. */
LSTM_API int lstm_status(lstm_handle *h);

/* Frees everything the handle owns (synchronises the device first).  NULL is accepted. */
LSTM_API int lstm_destroy(lstm_handle *h);

/* Reason of the last failure on this handle (or of the last failed lstm_create when h is NULL).
 * The string is owned by the library and valid until the next failing call. */
LSTM_API const char *lstm_last_error(const lstm_handle *h);

/*
 * Failure-path self-test.  The recurrent kernels hand h_t from CTA to CTA through stamped words and
 * every wait for such a word is bounded.  With cta >= 0, the recurrent kernel's CTA of that index
 * withholds its words in the following lstm_forward calls, so the waits of the other CTAs run out after
 * spin_limit clock ticks (spin_limit <= 0: the default limit, about a second): the kernel records
 * LSTM_ERR_TIMEOUT, stops waiting and runs to its end, and lstm_status returns the error with the CUDA
 * context intact.  cta < 0 restores normal operation.  Nothing faults or hangs in either mode.
 */
LSTM_API int lstm_selftest_timeout(lstm_handle *h, int cta, long long spin_limit);

/*
 * Measurement support.  With profiling on, lstm_forward brackets each of its kernels with CUDA events
 * on the launching stream; lstm_profile_read synchronises and returns, for the most recent
 * lstm_forward, per kernel kind k (LSTM_K_*): launches[k] and total device milliseconds ms[k].
 * Arrays must have LSTM_K_COUNT entries.
 */
enum { LSTM_K_STAGE = 0, LSTM_K_PROJ = 1, LSTM_K_RECUR = 2, LSTM_K_COUNT = 3 };
LSTM_API int lstm_profile_enable(lstm_handle *h, int on);
LSTM_API int lstm_profile_read(lstm_handle *h, int *launches, float *ms);

/*
 * Step-cost probe of the register-resident recurrent kernel (bf16 dense LSTM handles, calls with one sequence;
 * calls with more run normally).  A recurrent step is a chain: wait for the other CTAs' h words -> tensor-core products ->
 * CTA barrier, reduction, gate functions -> publish.  With a non-zero mask the following lstm_forward calls
 * leave parts of that chain out, so that timing them shows what each part costs (the "empty step": exchange
 * only, is the floor no kernel of this structure can go below).  Bits: LSTM_PROBE_NO_PRODUCTS (no tensor
 * instructions), LSTM_PROBE_NO_GATES (no reduction, gate functions or output stores; every unit still
 * publishes a word per step), LSTM_PROBE_NO_EXCHANGE (no waiting for other CTAs), LSTM_PROBE_WHOLE_STEP (nothing left
 * out: the measurement build itself, with the projection as a launch of its own, as the yardstick the other modes
 * are compared with; its outputs are valid).  With any other bit OUTPUTS ARE UNDEFINED
 * while a mask is set; 0 restores normal operation.  LSTM_ERR_UNSUPPORTED for handles that run another
 * recurrent kernel.  Every wait stays bounded in every mode.
 */
enum { LSTM_PROBE_NO_PRODUCTS = 1, LSTM_PROBE_NO_GATES = 2, LSTM_PROBE_NO_EXCHANGE = 4, LSTM_PROBE_WHOLE_STEP = 8 };
LSTM_API int lstm_probe(lstm_handle *h, int parts_left_out);

/*
 * Read-only facts about how the handle runs (for reports): writes up to n values into out and
 * returns the number available.  Order: [0] SM count, [1] CTAs of the recurrent kernel per direction,
 * [2] threads per CTA, [3] dynamic shared memory bytes per CTA at max_B, [4] recurrent-matrix rows
 * resident in shared memory per CTA (max over CTAs), [5] rows streamed from L2 per CTA (max),
 * [6] split-K factor of the input projection at max_T*max_B, [7] 1 if the projection uses the tensor-core
 * (tcgen05) kernel, [8] kernels launched by the most recent lstm_forward (before the first call: the count expected),
 * [9] 1 if the recurrence keeps its weights in registers (bf16 dense), 0 for the shared-memory kernel,
 * [10] 16-column weight tiles per warp held in registers, [11] per warp held in shared memory,
 * [12] nonzero if a call at max_B runs the batched tensor-core (tcgen05) recurrence (2: as clusters of two CTAs
 * that split K, 1: every CTA on its own): bf16 dense LSTM handles use
 * it for batches of 5 to 64 sequences where its operand ring fits beside the resident slice, and the
 * register-resident kernel (passes of four sequences) otherwise,
 * [13] 1 if a CSR handle runs the register-resident sparse kernel (bf16 storage, at most 16 units per CTA,
 * lane lists short enough for registers), 0 for the shared-memory CSR kernel, [14] its entry slots per lane,
 * [15] shared-memory wavefronts per step and CTA that its gathers lose to bank conflicts (worst CTA),
 * [16] the compact width when the handle runs a row/column-pruned stack on its surviving units only (0: it does
 * not; then [0]..[15] describe the handle itself, otherwise the inner handle of that width), [17] the number
 * of (layer, direction, unit) triples removed, [18] 1 if calls with up to four sequences run the layer-wavefront
 * kernel (unidirectional bf16 dense stacks of 2 to 4 layers whose slices fit on-chip with the SMs split between
 * the layers: all layers in one launch, layer l on timestep t beside layer l-1 on t+1).
 */
LSTM_API int lstm_info(const lstm_handle *h, int64_t *out, int n);

/*
 * Latency hysteresis (Section 3): on a measured latency-versus-size curve a size is a latency hysteresis
 * point (LHP) when no LARGER size runs within (1 + eps) of its latency; every other size is dominated
 * (a larger model is at least as fast) and the share of dominated sizes is the paper's architecture-space
 * redundancy.  Host arrays, no GPU work:
 *   sizes[n] distinct positive sizes in any order, latency[n] > 0 in any one unit, eps >= 0 the relative
 *   timing noise below which two latencies count as equal.
 * lstm_lhp_points writes is_lhp[i] in {0,1} and, if count is not NULL, the number of LHPs.
 * lstm_nearest_lhp returns in *out_size the smallest LHP >= requested (the size a pruned model is grown
 * back to, step (c) of Section 5.1); LSTM_ERR_UNSUPPORTED when requested exceeds every measured size.
 * Both return LSTM_ERR_INVALID for NULL arrays, n <= 0, eps < 0, a non-positive or non-finite latency, or
 * a repeated size.
 */
LSTM_API int lstm_lhp_points(const int *sizes, const double *latency, int n, double eps, int *is_lhp, int *count);
LSTM_API int lstm_nearest_lhp(const int *sizes, const double *latency, int n, double eps, int requested, int *out_size);

/*
 * Folds a per-feature affine map on a layer's INPUT into that layer's input weights (Section 5.2 uses
 * batch normalisation between recurrent layers; with its statistics frozen it is x' = scale * x + shift
 * per feature, scale = gamma / sqrt(var + epsilon), shift = beta - mean * scale):
 *     Wx (scale * x + shift) + b  =  (Wx diag(scale)) x + (b + Wx shift)
 * Host arrays: wx [rows, cols] row-major, b [rows] or NULL (zeros), scale, shift [cols] (either may be
 * NULL: ones / zeros); writes wx_out [rows, cols] (may be wx itself) and b_out [rows] (may be b itself).
 * The bias sum is accumulated in double.  Apply it to each (layer, direction) that reads normalised
 * input, before lstm_create; the pruning mask, if any, applies to the folded matrix unchanged.
 * Returns LSTM_ERR_INVALID for NULL wx / outputs or non-positive sizes.
 */
LSTM_API int lstm_fold_input_affine(const float *wx, const float *b, int rows, int cols, const float *scale,
                                    const float *shift, float *wx_out, float *b_out);

/*
 * Create-time layout of one pruned recurrent matrix for the register-resident sparse kernel (Section 4: the
 * mask-based scheme leaves an unstructured pattern of surviving weights), as a host-only call so that the
 * layout can be inspected and tested without a GPU; lstm_create runs the same code.
 *   rowptr/col/val: CSR of Wh [4*hidden x hidden], rows in gate-block order q*hidden + j, columns increasing.
 *   The hidden units are split evenly over `ctas` CTAs of `warps` (8 or 16) warps; warp w owns the columns
 *   [w*kspan, (w+1)*kspan) (kspan a multiple of 32 with warps*kspan >= hidden); inside a warp every lane owns
 *   at most two of the CTA's 4*units rows, longest rows dealt first.
 * Outputs (each may be NULL): *longest = entries of the longest lane list; rows[ctas*warps*32] = the lanes' two
 * local rows (4*unit + gate in byte 0 and byte 1, 0xff = none); entries[ctas*warps*slots*32] = the lists padded to
 * `slots` (>= *longest) words {bf16 value:16 | second-row flag:1 | 4*(column - w*kspan):15}, stored
 * [cta][warp][slot][lane], ordered so that the 32 gathers of a slot fall into different shared-memory banks
 * where the pattern allows; *conflict_wavefronts = extra wavefronts per step that remain (worst CTA).
 * LSTM_ERR_UNSUPPORTED when a CTA would own more than `warps` units; LSTM_ERR_INVALID for bad arguments.
 */
LSTM_API int lstm_csr_lane_layout(const int32_t *rowptr, const int32_t *col, const float *val, int hidden, int ctas,
                                  int warps, int kspan, int slots, uint32_t *entries, uint32_t *rows, int *longest,
                                  long long *conflict_wavefronts);

/*
 * Forward pass without any allocation (the paper has no counterpart: this exists for deployment).
 * For callers that cannot allocate device memory at call time or at all -- a serving loop whose memory
 * pool is fixed at start-up, a host framework whose allocator owns the device, a process that must not
 * grow after initialisation -- and therefore cannot use lstm_create, which allocates packed weights and
 * a workspace.  One layer, one direction, fp32, dense; every tensor is the caller's:
 *   wx [4H, in_dim], wh [4H, H] row-major fp32 and b [4H] (or NULL = zeros), gate row blocks i,f,g,o;
 *   x [T,B,in_dim]; h0, c0 [B,H] or NULL (zeros); y [T,B,H]; hT, cT [B,H] or NULL (not wanted).
 * All are DEVICE pointers and are only read (wx, wh, b, x, h0, c0) or written (y, hT, cT) by this call.
 * The same cell equations and arithmetic as a LSTM_F32 handle (fp64 sums and gate functions, fp32
 * storage); weights are read through L2 every step
 * (nothing is packed or kept on-chip), so this path is slower than a handle.
 * Scratch: the per-step exchange words and a status word live in a fixed array inside the library
 * image (about 128 KiB of device memory on every GPU that loads the library, held until exit).
 * Limits: B * hidden <= LSTM_NOALLOC_MAX_BH and B * (in_dim + hidden + hidden/SMs + 1) floats must fit
 * in one CTA's shared memory; beyond them the call returns LSTM_ERR_UNSUPPORTED and launches nothing.
 * The first call on a device (with that device current) looks up the array's device address and the
 * device limits; make that first call before any stream capture.  Every call clears the array and then
 * uses it: calls that overlap on the same GPU (two streams, two threads) race on it and must be
 * serialised by the caller.  The call calls no cudaMalloc / cudaFree or any allocating routine; it
 * enqueues on cuda_stream and synchronises that stream before returning, so a device-side timeout of
 * this very call is returned as LSTM_ERR_TIMEOUT.
 * err (may be NULL): caller-owned buffer of errlen bytes that receives the reason of a failure.
 * Failure-path self-test: with LSTM_B200_NOALLOC_SELFTEST=<cta>:<clock ticks> in the environment, that CTA withholds
 * its exchange words, the other CTAs' bounded waits run out after the given ticks, and the call returns
 * LSTM_ERR_TIMEOUT with the CUDA context intact (nothing faults or hangs); the next call without it is normal again.
 */
#define LSTM_NOALLOC_MAX_BH 8192
LSTM_API int lstm_forward_noalloc(const float *wx, const float *wh, const float *b, int in_dim, int hidden,
                         const float *x, int T, int B, const float *h0, const float *c0,
                         float *y, float *hT, float *cT, void *cuda_stream, char *err, int errlen);

#ifdef __cplusplus
}
#endif
#endif /* LSTM_B200_H */
