// Create-time layout of a pruned recurrent matrix for the register-resident sparse kernel (host code).
#pragma once
#include <cstdint>
#include <cstring>
#include <vector>

namespace lstm {

inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);   // NaN stays NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
inline float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

// Entry lists of one (layer, direction): lists[(cta * nw + warp) * 32 + lane] holds the words
// {bf16 value : 16 | second-row flag : 1 | 4 * column inside the warp's range : 15} of that lane, rows[same index]
// its two local rows (byte 0, byte 1; 0xff = none).
struct CsrLaneLists {
    std::vector<std::vector<unsigned>> lists;
    std::vector<unsigned> rows;
    int longest = 0;            // entries of the longest list
};

// rowptr/col/val: CSR of the recurrent matrix [4H x H] with rows in gate-block order q * H + j.  The H units are
// split evenly over ncta CTAs; warp w of a CTA owns columns [w * kspan, (w + 1) * kspan).  Rows are dealt to the
// lanes of each warp longest-first (at most two per lane; needs 4 * units per CTA <= 64).
void csr_lane_lists(const int *rowptr, const int *col, const float *val, int H, int ncta, int nw, int kspan, CsrLaneLists &out);

// Packs the lists into [cta][warp][slots][32 lanes] words for a kernel built with `slots` entry slots per lane
// (slots >= longest).  Within a warp the entries of the 32 lanes are ordered so that the shared-memory gathers
// of one slot hit different banks wherever the pattern allows; free slots are filled with zero-valued words
// that point at unused banks.  *conflict_wavefronts (optional) receives the number of extra shared-memory
// wavefronts per step and CTA that remain, summed over warps, maximum over CTAs.
std::vector<unsigned> csr_pack_slots(const CsrLaneLists &in, int ncta, int nw, int slots, int kspan, long long *conflict_wavefronts);

}  // namespace lstm
