/*
 * fp64 CPU oracle for the stacked (optionally bidirectional) LSTM inference forward pass.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the yardstick the CUDA library is compared with. It shares
 * no code, header, table or build target with the CUDA path, and nothing in the product may call it.
 *
 * What it computes: the paper's cell equations (Section 4, the unnumbered equation block that defines
 * f_t, i_t, o_t, g_t, c_t, h_t) with H* = zero hidden layers inside each gate, i.e. the conventional
 * LSTM that the paper uses as its baseline (Section 5.1: two stacked layers; Section 5.2: bidirectional
 * DeepSpeech2 stack).  With W = [Wx | Wh] acting on the concatenation [x_t, h_{t-1}]:
 *
 *     z_q[j] = b_q[j] + sum_k Wx_q[j,k] * x_t[k] + sum_k Wh_q[j,k] * h_{t-1}[k]        q in {i,f,g,o}
 *     i = sigma(z_i)  f = sigma(z_f)  g = tanh(z_g)  o = sigma(z_o)        sigma(z) = 1/(1+exp(-z))
 *     c_t = f * c_{t-1} + i * g            h_t = o * tanh(c_t)
 *
 * Masks follow Section 4 ("mask-based approach"): the effective weight is W (x) Msk, so a masked entry
 * is an explicit zero.  Two walks over the same weights are kept: a dense walk that multiplies every
 * entry by its mask bit, and a CSR walk that visits the surviving entries only.
 *
 * Conventions (choices the paper leaves open):
 *   - gate rows are packed in blocks of H rows in the order i, f, g, o (row q*H + j is gate q, unit j);
 *   - one bias vector per gate;
 *   - a bidirectional layer's output is the concatenation [forward | reverse]; the reverse direction
 *     processes t = T-1 .. 0, stores its output for position t at y[t], and its final state is the one
 *     after t = 0;
 *   - state index for (layer l, direction d) is l*D + d.
 *
 * Arithmetic: everything in double; every sum runs sequentially in index order k = 0,1,2,...;
 * std exp / tanh.  Weights arrive as float (already rounded by the caller to whatever the device
 * stores) and are widened exactly.  OpenMP only distributes independent outputs (b, j) over threads;
 * no sum is split, so the result does not depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    /* dense description (used when the matching rowptr is NULL) */
    const float   *wx;      /* [4H, in_l] row-major */
    const float   *wh;      /* [4H, H]   row-major */
    const float   *b;       /* [4H] or NULL = zeros */
    const uint8_t *mask_x;  /* [4H, in_l], 1 = keep, or NULL = all kept */
    const uint8_t *mask_h;  /* [4H, H] or NULL */
    /* CSR description (rowptr int32[4H+1], col int32[nnz], val float[nnz]) */
    const int32_t *wx_rowptr, *wx_col; const float *wx_val;
    const int32_t *wh_rowptr, *wh_col; const float *wh_val;
} oracle_weights;

static double sigma(double z) { return 1.0 / (1.0 + exp(-z)); }

/* sum_k M[row,k] * v[k] added onto acc, entries in index order; dense-with-mask or CSR walk */
static double add_row_product(double acc, int row, int ncol, const float *dense, const uint8_t *mask,
                              const int32_t *rowptr, const int32_t *col, const float *val,
                              const double *v)
{
    if (rowptr) {
        for (int32_t e = rowptr[row]; e < rowptr[row + 1]; ++e)
            acc += (double)val[e] * v[col[e]];
    } else {
        const float *r = dense + (size_t)row * ncol;
        const uint8_t *m = mask ? mask + (size_t)row * ncol : NULL;
        for (int k = 0; k < ncol; ++k) {
            double w = (double)r[k];
            if (m) w = w * (double)m[k];          /* W (x) Msk: a masked weight is an explicit zero */
            acc += w * v[k];
        }
    }
    return acc;
}

/* One layer, one direction, all timesteps. X is [T,B,in_l]; Y is [T,B,y_stride] written at y_off. */
static int run_direction(int in_l, int H, int T, int B, int reverse, const oracle_weights *w,
                         const double *X, const double *h0, const double *c0,
                         double *Y, int y_stride, int y_off, double *hT, double *cT)
{
    size_t n = (size_t)B * H;
    double *h_prev = (double *)calloc(n ? n : 1, sizeof(double));
    double *c_prev = (double *)calloc(n ? n : 1, sizeof(double));
    double *h_new  = (double *)calloc(n ? n : 1, sizeof(double));
    double *c_new  = (double *)calloc(n ? n : 1, sizeof(double));
    if (!h_prev || !c_prev || !h_new || !c_new) { free(h_prev); free(c_prev); free(h_new); free(c_new); return 1; }
    if (h0) memcpy(h_prev, h0, n * sizeof(double));
    if (c0) memcpy(c_prev, c0, n * sizeof(double));

    for (int s = 0; s < T; ++s) {
        int t = reverse ? T - 1 - s : s;
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(static)
#endif
        for (int b = 0; b < B; ++b) {
            for (int j = 0; j < H; ++j) {
                const double *x_t = X + ((size_t)t * B + b) * in_l;
                const double *h_p = h_prev + (size_t)b * H;
                double z[4];
                for (int q = 0; q < 4; ++q) {
                    int row = q * H + j;
                    double acc = w->b ? (double)w->b[row] : 0.0;
                    acc = add_row_product(acc, row, in_l, w->wx, w->mask_x,
                                          w->wx_rowptr, w->wx_col, w->wx_val, x_t);
                    acc = add_row_product(acc, row, H, w->wh, w->mask_h,
                                          w->wh_rowptr, w->wh_col, w->wh_val, h_p);
                    z[q] = acc;
                }
                double gi = sigma(z[0]);
                double gf = sigma(z[1]);
                double gg = tanh(z[2]);
                double go = sigma(z[3]);
                double c = gf * c_prev[(size_t)b * H + j] + gi * gg;
                double h = go * tanh(c);
                c_new[(size_t)b * H + j] = c;
                h_new[(size_t)b * H + j] = h;
                Y[((size_t)t * B + b) * y_stride + y_off + j] = h;
            }
        }
        double *tmp;
        tmp = h_prev; h_prev = h_new; h_new = tmp;
        tmp = c_prev; c_prev = c_new; c_new = tmp;
    }
    if (hT) memcpy(hT, h_prev, n * sizeof(double));
    if (cT) memcpy(cT, c_prev, n * sizeof(double));
    free(h_prev); free(c_prev); free(h_new); free(c_new);
    return 0;
}

/*
 * Whole stack.  w has L*D entries (index l*D + d, d = 1 is the reverse direction).
 * x [T,B,in_dim]; h0,c0 [L*D,B,H] or NULL (zeros); y [T,B,D*H]; hT,cT [L*D,B,H] or NULL.
 * Layer l > 0 reads the previous layer's [T,B,D*H] output.  Returns 0, or 1 on bad arguments /
 * allocation failure.
 */
int lstm_oracle_forward(int L, int D, int in_dim, int H, int T, int B, const oracle_weights *w,
                        const double *x, const double *h0, const double *c0,
                        double *y, double *hT, double *cT)
{
    if (L < 1 || (D != 1 && D != 2) || in_dim < 1 || H < 1 || T < 0 || B < 0 || !w || !y) return 1;
    if (T > 0 && B > 0 && !x) return 1;
    size_t out_n = (size_t)T * B * D * H;
    size_t st_n = (size_t)B * H;
    double *cur = NULL, *nxt = NULL;          /* inter-layer activations */
    if (L > 1) {
        cur = (double *)malloc((out_n ? out_n : 1) * sizeof(double));
        nxt = (double *)malloc((out_n ? out_n : 1) * sizeof(double));
        if (!cur || !nxt) { free(cur); free(nxt); return 1; }
    }
    const double *X = x;
    int in_l = in_dim;
    int rc = 0;
    for (int l = 0; l < L && !rc; ++l) {
        double *Y = (l == L - 1) ? y : nxt;
        for (int d = 0; d < D && !rc; ++d) {
            size_t s = (size_t)(l * D + d) * st_n;
            rc = run_direction(in_l, H, T, B, d == 1, &w[l * D + d], X,
                               h0 ? h0 + s : NULL, c0 ? c0 + s : NULL,
                               Y, D * H, d * H, hT ? hT + s : NULL, cT ? cT + s : NULL);
        }
        if (l < L - 1) { double *tmp = cur; cur = nxt; nxt = tmp; X = cur; in_l = D * H; }
    }
    free(cur); free(nxt);
    return rc;
}

/*
 * H-LSTM variant (paper, Section 4, same equation block with H* = ONE hidden layer inside each gate:
 * "hidden layer that performs a linear transformation followed by an activation function", here ReLU,
 * one of the internal activations the paper names).  For gate q in {i,f,g,o}, hidden width Hh:
 *
 *     r_q = relu(a_q + Ux_q x_t + Uh_q h_{t-1})                (Hh values; U_q = [Ux_q | Uh_q] acts on [x_t, h_{t-1}])
 *     z_q = b_q + W_q r_q                                       (H values)
 *     i = sigma(z_i)  f = sigma(z_f)  g = tanh(z_g)  o = sigma(z_o)   c_t = f c_{t-1} + i g   h_t = o tanh(c_t)
 *
 * Layout: ux [4Hh, in_l] and uh [4Hh, H] with row q*Hh + m; a [4Hh]; w [4H, Hh] with row q*H + j (block q
 * multiplies r_q); b [4H]; NULL biases are zeros.  Stacking, directions and state indexing as above.
 */
typedef struct {
    const float *ux, *uh, *a, *w, *b;
} oracle_hweights;

static int run_direction_h(int in_l, int H, int Hh, int T, int B, int reverse, const oracle_hweights *w,
                           const double *X, const double *h0, const double *c0,
                           double *Y, int y_stride, int y_off, double *hT, double *cT)
{
    size_t n = (size_t)B * H, nr = (size_t)B * 4 * Hh;
    double *h_prev = (double *)calloc(n ? n : 1, sizeof(double));
    double *c_prev = (double *)calloc(n ? n : 1, sizeof(double));
    double *h_new  = (double *)calloc(n ? n : 1, sizeof(double));
    double *c_new  = (double *)calloc(n ? n : 1, sizeof(double));
    double *r      = (double *)calloc(nr ? nr : 1, sizeof(double));
    if (!h_prev || !c_prev || !h_new || !c_new || !r) { free(h_prev); free(c_prev); free(h_new); free(c_new); free(r); return 1; }
    if (h0) memcpy(h_prev, h0, n * sizeof(double));
    if (c0) memcpy(c_prev, c0, n * sizeof(double));

    for (int s = 0; s < T; ++s) {
        int t = reverse ? T - 1 - s : s;
        /* hidden layers of the four gates */
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(static)
#endif
        for (int b = 0; b < B; ++b) {
            for (int m = 0; m < 4 * Hh; ++m) {
                const double *x_t = X + ((size_t)t * B + b) * in_l;
                const double *h_p = h_prev + (size_t)b * H;
                double acc = w->a ? (double)w->a[m] : 0.0;
                for (int k = 0; k < in_l; ++k) acc += (double)w->ux[(size_t)m * in_l + k] * x_t[k];
                for (int k = 0; k < H; ++k) acc += (double)w->uh[(size_t)m * H + k] * h_p[k];
                r[(size_t)b * 4 * Hh + m] = acc > 0.0 ? acc : 0.0;
            }
        }
        /* gate pre-activations from the hidden layers, gates, state update */
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(static)
#endif
        for (int b = 0; b < B; ++b) {
            for (int j = 0; j < H; ++j) {
                double z[4];
                for (int q = 0; q < 4; ++q) {
                    int row = q * H + j;
                    const double *rq = r + (size_t)b * 4 * Hh + (size_t)q * Hh;
                    double acc = w->b ? (double)w->b[row] : 0.0;
                    for (int m = 0; m < Hh; ++m) acc += (double)w->w[(size_t)row * Hh + m] * rq[m];
                    z[q] = acc;
                }
                double gi = sigma(z[0]);
                double gf = sigma(z[1]);
                double gg = tanh(z[2]);
                double go = sigma(z[3]);
                double c = gf * c_prev[(size_t)b * H + j] + gi * gg;
                double h = go * tanh(c);
                c_new[(size_t)b * H + j] = c;
                h_new[(size_t)b * H + j] = h;
                Y[((size_t)t * B + b) * y_stride + y_off + j] = h;
            }
        }
        double *tmp;
        tmp = h_prev; h_prev = h_new; h_new = tmp;
        tmp = c_prev; c_prev = c_new; c_new = tmp;
    }
    if (hT) memcpy(hT, h_prev, n * sizeof(double));
    if (cT) memcpy(cT, c_prev, n * sizeof(double));
    free(h_prev); free(c_prev); free(h_new); free(c_new); free(r);
    return 0;
}

int hlstm_oracle_forward(int L, int D, int in_dim, int H, int Hh, int T, int B, const oracle_hweights *w,
                         const double *x, const double *h0, const double *c0,
                         double *y, double *hT, double *cT)
{
    if (L < 1 || (D != 1 && D != 2) || in_dim < 1 || H < 1 || Hh < 1 || T < 0 || B < 0 || !w || !y) return 1;
    if (T > 0 && B > 0 && !x) return 1;
    for (int i = 0; i < L * D; ++i) if (!w[i].ux || !w[i].uh || !w[i].w) return 1;
    size_t out_n = (size_t)T * B * D * H;
    size_t st_n = (size_t)B * H;
    double *cur = NULL, *nxt = NULL;
    if (L > 1) {
        cur = (double *)malloc((out_n ? out_n : 1) * sizeof(double));
        nxt = (double *)malloc((out_n ? out_n : 1) * sizeof(double));
        if (!cur || !nxt) { free(cur); free(nxt); return 1; }
    }
    const double *X = x;
    int in_l = in_dim;
    int rc = 0;
    for (int l = 0; l < L && !rc; ++l) {
        double *Y = (l == L - 1) ? y : nxt;
        for (int d = 0; d < D && !rc; ++d) {
            size_t s = (size_t)(l * D + d) * st_n;
            rc = run_direction_h(in_l, H, Hh, T, B, d == 1, &w[l * D + d], X,
                                 h0 ? h0 + s : NULL, c0 ? c0 + s : NULL,
                                 Y, D * H, d * H, hT ? hT + s : NULL, cT ? cT + s : NULL);
        }
        if (l < L - 1) { double *tmp = cur; cur = nxt; nxt = tmp; X = cur; in_l = D * H; }
    }
    free(cur); free(nxt);
    return rc;
}

int lstm_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
