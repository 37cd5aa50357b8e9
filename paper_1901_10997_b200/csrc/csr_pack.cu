// Create-time layout of a pruned recurrent matrix for the register-resident sparse kernel: which lane of which
// warp keeps which surviving weights (Section 4 of the paper: the mask-based scheme leaves an unstructured
// pattern, about one weight in ten or twenty), and in which order it walks them.
#include <algorithm>
#include <cstring>
#include <numeric>

#include "csr_pack.h"

namespace lstm {

void csr_lane_lists(const int *rowptr, const int *col, const float *val, int H, int ncta, int nw, int kspan, CsrLaneLists &out)
{
    out.lists.assign((size_t)ncta * nw * 32, {});
    out.rows.assign((size_t)ncta * nw * 32, 0xffffu);
    out.longest = 0;
    const int base = H / ncta, rem = H % ncta;
    std::vector<int> cnt, order, load(32), second(32);
    for (int c = 0; c < ncta; ++c) {
        const int nu = base + (c < rem ? 1 : 0), u0 = c * base + std::min(c, rem);
        const int R = 4 * nu;                                  // local row r = 4 * unit + gate
        for (int w = 0; w < nw; ++w) {
            const int k0 = w * kspan, k1 = std::min(H, k0 + kspan);
            if (k0 >= H && R == 0) continue;
            // entries of every local row inside this warp's column range (columns are sorted inside a row)
            cnt.assign(R, 0);
            std::vector<std::pair<int, int>> span(R);         // [first, last) entry index of the row in this range
            for (int r = 0; r < R; ++r) {
                const int grow = (r & 3) * H + u0 + (r >> 2);
                const int *b = col + rowptr[grow], *e = col + rowptr[grow + 1];
                const int *lo = std::lower_bound(b, e, k0), *hi = std::lower_bound(lo, e, k1);
                span[r] = {(int)(lo - col), (int)(hi - col)};
                cnt[r] = (int)(hi - lo);
            }
            order.resize(R);
            std::iota(order.begin(), order.end(), 0);
            std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return cnt[x] > cnt[y]; });
            std::fill(load.begin(), load.end(), 0);
            std::fill(second.begin(), second.end(), 0);
            const size_t lbase = (size_t)(c * nw + w) * 32;
            auto put = [&](int lane, int r, bool is_second) {
                std::vector<unsigned> &L = out.lists[lbase + lane];
                for (int e = span[r].first; e < span[r].second; ++e)
                    L.push_back(((unsigned)f32_to_bf16_rne(val[e]) << 16) | (is_second ? 0x8000u : 0u) | ((unsigned)(col[e] - k0) << 2));
                unsigned &rw = out.rows[lbase + lane];
                rw = is_second ? ((rw & 0x00ffu) | ((unsigned)r << 8)) : ((rw & 0xff00u) | (unsigned)r);
                load[lane] += cnt[r];
            };
            for (int i = 0; i < R && i < 32; ++i) put(i, order[i], false);
            for (int i = 32; i < R; ++i) {                    // the shorter rows join the lanes with the least work
                int best = -1;
                for (int l = 0; l < 32; ++l)
                    if (!second[l] && (best < 0 || load[l] < load[best])) best = l;
                put(best, order[i], true);
                second[best] = 1;
            }
            for (int l = 0; l < 32; ++l) out.longest = std::max(out.longest, load[l]);
        }
    }
}

std::vector<unsigned> csr_pack_slots(const CsrLaneLists &in, int ncta, int nw, int slots, int kspan, long long *conflict_wavefronts)
{
    std::vector<unsigned> packed((size_t)ncta * nw * slots * 32, 0u);
    long long worst = 0;
    std::vector<unsigned> rest[32];
    for (int c = 0; c < ncta; ++c) {
        long long extra_cta = 0;
        for (int w = 0; w < nw; ++w) {
            const size_t lbase = (size_t)(c * nw + w) * 32;
            int pads[32], lanes[32];
            for (int l = 0; l < 32; ++l) {
                rest[l] = in.lists[lbase + l];
                pads[l] = slots - (int)rest[l].size();
                lanes[l] = l;
            }
            // lanes with the least slack choose first
            std::stable_sort(lanes, lanes + 32, [&](int x, int y) { return pads[x] < pads[y]; });
            unsigned *dst = packed.data() + (size_t)(c * nw + w) * slots * 32;
            for (int e = 0; e < slots; ++e) {
                int bank_use[32] = {0};
                int bank_col[32];
                bool padded[32] = {false};
                std::fill(bank_col, bank_col + 32, -1);
                for (int li = 0; li < 32; ++li) {
                    const int l = lanes[li];
                    std::vector<unsigned> &R = rest[l];
                    if (R.empty()) { padded[l] = true; continue; }
                    // an entry whose bank is free in this slot (or that repeats a column already read: a broadcast)
                    int pick = -1, pick_cost = 1 << 30;
                    for (int i = 0; i < (int)R.size(); ++i) {
                        const int cl = (int)((R[i] & 0x7fffu) >> 2), bk = cl & 31;
                        const int cost = (bank_use[bk] == 0 || bank_col[bk] == cl) ? 0 : bank_use[bk];
                        if (cost < pick_cost) { pick_cost = cost; pick = i; if (cost == 0) break; }
                    }
                    if (pick_cost > 0 && pads[l] > 0) { --pads[l]; padded[l] = true; continue; }
                    const unsigned word = R[pick];
                    R[pick] = R.back();
                    R.pop_back();
                    const int cl = (int)((word & 0x7fffu) >> 2), bk = cl & 31;
                    if (!(bank_use[bk] > 0 && bank_col[bk] == cl)) ++bank_use[bk];
                    if (bank_col[bk] < 0) bank_col[bk] = cl;
                    dst[(size_t)e * 32 + l] = word;
                }
                // zero-valued words for the lanes that sit this slot out, each on a bank nobody reads
                int free_bank = 0;
                for (int l = 0; l < 32; ++l) {
                    if (!padded[l]) continue;
                    while (free_bank < 32 && bank_use[free_bank] > 0) ++free_bank;
                    const int bk = free_bank < 32 ? free_bank++ : 0;
                    dst[(size_t)e * 32 + l] = (unsigned)std::min(bk, kspan - 1) << 2;
                }
                int deepest = 1;
                for (int b = 0; b < 32; ++b) deepest = std::max(deepest, bank_use[b]);
                extra_cta += deepest - 1;
            }
        }
        worst = std::max(worst, extra_cta);
    }
    if (conflict_wavefronts) *conflict_wavefronts = worst;
    return packed;
}

}  // namespace lstm
