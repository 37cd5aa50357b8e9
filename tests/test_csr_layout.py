"""Create-time layout of a pruned recurrent matrix for the register-resident sparse kernel (host code, no GPU).

The layout must hold every surviving weight exactly once, in the lane that owns its row and the warp that
owns its column, with the value rounded to bf16; what it adds (row dealing, slot order, padding) may change
the order of the work but never the matrix."""
import numpy as np
import pytest

import lstm_workloads as wl


def _csr(w, mask):
    rp = [0]
    cols, vals = [], []
    for r in range(w.shape[0]):
        k = np.nonzero(mask[r])[0]
        cols.extend(k.tolist())
        vals.extend(w[r, k].tolist())
        rp.append(len(cols))
    return np.array(rp, np.int32), np.array(cols, np.int32), np.array(vals, np.float32)


def _rebuild(entries, rows, H, ctas, warps, kspan):
    """Dense [4H, H] matrix from the packed words."""
    out = np.zeros((4 * H, H), np.float64)
    seen = np.zeros((4 * H, H), np.int32)
    base, rem = divmod(H, ctas)
    for c in range(ctas):
        nu = base + (1 if c < rem else 0)
        u0 = c * base + min(c, rem)
        for w in range(warps):
            for lane in range(32):
                rw = int(rows[c, w, lane])
                local = (rw & 0xff, (rw >> 8) & 0xff)
                for word in entries[c, w, :, lane]:
                    word = int(word)
                    val = np.array([word & 0xffff0000], np.uint32).view(np.float32)[0]
                    if val == 0.0:
                        continue                      # padding (or a kept weight that is exactly zero: contributes nothing)
                    r = local[1 if word & 0x8000 else 0]
                    assert r != 0xff and r < 4 * nu
                    k = w * kspan + ((word & 0x7fff) >> 2)
                    assert k < H
                    grow = (r & 3) * H + u0 + (r >> 2)
                    out[grow, k] = val
                    seen[grow, k] += 1
    return out, seen


@pytest.mark.parametrize("H,ctas,warps,density", [(300, 148, 8, 0.3), (1500, 148, 16, 0.10), (640, 74, 16, 0.05), (97, 97, 8, 0.5)])
def test_layout_holds_every_surviving_weight_once(H, ctas, warps, density):
    import paper_1901_10997_b200 as pkg
    rng = np.random.default_rng(H)
    w = wl.round_to_bf16(rng.uniform(-0.1, 0.1, size=(4 * H, H)).astype(np.float32))
    w[w == 0] = 0.0625
    mask = rng.random((4 * H, H)) < density
    mask[5] = False                                    # an empty row
    rp, col, val = _csr(w, mask)
    kspan = -(-(-(-H // warps)) // 32) * 32
    rc, longest, rows, _e, _c = pkg.lstm_csr_lane_layout(rp, col, val, H, ctas, warps, kspan)
    assert rc == pkg.LSTM_OK and longest > 0
    slots = -(-longest // 8) * 8
    rc, longest2, rows, entries, conflicts = pkg.lstm_csr_lane_layout(rp, col, val, H, ctas, warps, kspan, slots)
    assert rc == pkg.LSTM_OK and longest2 == longest
    got, seen = _rebuild(entries, rows, H, ctas, warps, kspan)
    assert np.array_equal(seen > 0, mask)
    assert seen.max() == 1
    assert np.array_equal(got, np.where(mask, w, 0.0).astype(np.float64))
    # every local row of a CTA is owned by exactly one lane in every warp
    base, rem = divmod(H, ctas)
    for c in (0, ctas - 1):
        nu = base + (1 if c < rem else 0)
        for wp in range(warps):
            owned = []
            for lane in range(32):
                rw = int(rows[c, wp, lane])
                owned += [r for r in (rw & 0xff, (rw >> 8) & 0xff) if r != 0xff]
            assert sorted(owned) == list(range(4 * nu))
    # dealing rows longest-first: a lane with two rows got two SHORT ones, so the longest list is about the longest
    # single row piece (one row inside one warp's column range), not two of them
    pieces = np.add.reduceat(mask.astype(np.int32), np.arange(0, H, kspan), axis=1)
    upc = -(-H // ctas)
    assert longest >= pieces.max()
    assert longest <= (pieces.max() if 4 * upc <= 32 else 1.25 * pieces.max() + 2)


def test_slot_order_removes_most_bank_conflicts():
    """The gathers of one slot read 32 staged h values; ordered as they come (by column) many of them share a
    shared-memory bank.  The create-time order must leave fewer extra wavefronts than the natural order."""
    import paper_1901_10997_b200 as pkg
    H, ctas, warps, density = 1500, 148, 16, 0.10
    rng = np.random.default_rng(7)
    w = wl.round_to_bf16(rng.uniform(-0.1, 0.1, size=(4 * H, H)).astype(np.float32))
    mask = rng.random((4 * H, H)) < density
    rp, col, val = _csr(w, mask)
    kspan = 96
    rc, longest, rows, _e, _c = pkg.lstm_csr_lane_layout(rp, col, val, H, ctas, warps, kspan)
    slots = -(-longest // 8) * 8
    rc, _l, rows, entries, conflicts = pkg.lstm_csr_lane_layout(rp, col, val, H, ctas, warps, kspan, slots)
    assert rc == pkg.LSTM_OK
    # natural order: every lane walks its entries sorted by column; count the extra wavefronts of CTA 0
    natural = 0
    for wp in range(warps):
        lists = []
        for lane in range(32):
            ws = [int(x) for x in entries[0, wp, :, lane] if (int(x) & 0xffff0000)]
            lists.append(sorted(ws, key=lambda x: x & 0x7fff))
        for e in range(max(len(l) for l in lists)):
            banks = {}
            for l in lists:
                if e < len(l):
                    c = (l[e] & 0x7fff) >> 2
                    banks.setdefault(c & 31, set()).add(c)
            natural += max(len(v) for v in banks.values()) - 1
    assert conflicts < 0.5 * natural, (conflicts, natural)


def test_layout_rejects_what_the_kernel_cannot_hold():
    import paper_1901_10997_b200 as pkg
    rp = np.zeros(4 * 40 + 1, np.int32)
    z = np.zeros(1, np.int32)
    rc, *_ = pkg.lstm_csr_lane_layout(rp, z, z.astype(np.float32), 40, 2, 16, 32)       # 20 units per CTA > 16 warps
    assert rc == pkg.LSTM_ERR_UNSUPPORTED
    rc, *_ = pkg.lstm_csr_lane_layout(rp, z, z.astype(np.float32), 40, 40, 16, 48)      # kspan not a multiple of 32
    assert rc == pkg.LSTM_ERR_INVALID
