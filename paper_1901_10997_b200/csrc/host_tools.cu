// Host-side helpers of the library that run no kernel: the latency-hysteresis analysis of a measured
// latency-versus-size curve (paper, Section 3) and the folding of an inter-layer affine map into the
// next layer's input weights (paper, Section 5.2: batch normalisation between recurrent layers, which at
// inference time is a fixed scale and shift per feature).
#include "../../include/lstm_b200.h"
#include "csr_pack.h"

#include <algorithm>
#include <cmath>
#include <limits>
#include <vector>

namespace {

// flags[i] = 1 when point i is a latency hysteresis point: no larger size runs within (1 + eps) of its latency
bool mark_lhps(const int *sizes, const double *latency, int n, double eps, std::vector<int> &flags)
{
    if (!sizes || !latency || n <= 0 || !(eps >= 0.0)) return false;
    flags.assign(n, 0);
    for (int i = 0; i < n; ++i) {
        if (sizes[i] <= 0 || !(latency[i] > 0.0) || !std::isfinite(latency[i])) return false;
        for (int j = 0; j < i; ++j)
            if (sizes[j] == sizes[i]) return false;
    }
    for (int i = 0; i < n; ++i) {
        double best_larger = std::numeric_limits<double>::infinity();
        for (int j = 0; j < n; ++j)
            if (sizes[j] > sizes[i] && latency[j] < best_larger) best_larger = latency[j];
        flags[i] = latency[i] * (1.0 + eps) < best_larger ? 1 : 0;
    }
    return true;
}

}  // namespace

extern "C" {

int lstm_lhp_points(const int *sizes, const double *latency, int n, double eps, int *is_lhp, int *count)
{
    std::vector<int> flags;
    if (!is_lhp || !mark_lhps(sizes, latency, n, eps, flags)) return LSTM_ERR_INVALID;
    int c = 0;
    for (int i = 0; i < n; ++i) { is_lhp[i] = flags[i]; c += flags[i]; }
    if (count) *count = c;
    return LSTM_OK;
}

int lstm_nearest_lhp(const int *sizes, const double *latency, int n, double eps, int requested, int *out_size)
{
    std::vector<int> flags;
    if (!out_size || !mark_lhps(sizes, latency, n, eps, flags)) return LSTM_ERR_INVALID;
    int best = -1;
    for (int i = 0; i < n; ++i)
        if (flags[i] && sizes[i] >= requested && (best < 0 || sizes[i] < best)) best = sizes[i];
    if (best < 0) return LSTM_ERR_UNSUPPORTED;      // the request is larger than every measured size
    *out_size = best;
    return LSTM_OK;
}

int lstm_fold_input_affine(const float *wx, const float *b, int rows, int cols, const float *scale, const float *shift,
                           float *wx_out, float *b_out)
{
    if (!wx || !wx_out || !b_out || rows <= 0 || cols <= 0) return LSTM_ERR_INVALID;
    for (int r = 0; r < rows; ++r) {
        const float *src = wx + (size_t)r * cols;
        float *dst = wx_out + (size_t)r * cols;
        double acc = b ? (double)b[r] : 0.0;
        for (int k = 0; k < cols; ++k) {
            const float w = src[k];
            if (shift) acc += (double)w * (double)shift[k];
            dst[k] = scale ? w * scale[k] : w;
        }
        b_out[r] = (float)acc;
    }
    return LSTM_OK;
}

}  // extern "C"


// The create-time layout of one pruned recurrent matrix for the register-resident sparse kernel, exposed so
// that it can be inspected without a GPU (see the header).
extern "C" int lstm_csr_lane_layout(const int32_t *rowptr, const int32_t *col, const float *val, int hidden, int ctas,
                                    int warps, int kspan, int slots, uint32_t *entries, uint32_t *rows, int *longest,
                                    long long *conflict_wavefronts)
{
    if (!rowptr || hidden < 1 || ctas < 1 || ctas > hidden || (warps != 8 && warps != 16) || kspan < 32 || (kspan % 32) != 0 ||
        kspan * 4 > 0x7ffc || (long long)kspan * warps < hidden || slots < 0)
        return LSTM_ERR_INVALID;
    if ((hidden + ctas - 1) / ctas > warps) return LSTM_ERR_UNSUPPORTED;      // more than 4 * warps rows per CTA
    if (rowptr[4 * hidden] > 0 && (!col || !val)) return LSTM_ERR_INVALID;
    lstm::CsrLaneLists lists;
    lstm::csr_lane_lists(rowptr, col, val, hidden, ctas, warps, kspan, lists);
    if (longest) *longest = lists.longest;
    if (rows) std::copy(lists.rows.begin(), lists.rows.end(), rows);
    if (entries) {
        if (slots < lists.longest) return LSTM_ERR_INVALID;
        const std::vector<unsigned> packed = lstm::csr_pack_slots(lists, ctas, warps, slots, kspan, conflict_wavefronts);
        std::copy(packed.begin(), packed.end(), entries);
    }
    return LSTM_OK;
}
