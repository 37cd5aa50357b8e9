"""Pins of the fp64 oracle against things other than itself (CPU only).

The paper (Section 4, cell equations) prints no worked numeric example, so the oracle is pinned by
closed forms, a hand-evaluated single-unit sequence, a brute-force recursive evaluation on tiny
inputs, structural invariants, a library special case (the conventional LSTM routine of PyTorch on
CPU in float64) and a mutation check showing that planted mistakes are caught.
"""
import math
import shutil
import subprocess
import ctypes
from functools import lru_cache
from pathlib import Path

import numpy as np
import pytest

import lstm_workloads as wl

GOLDEN = Path(__file__).resolve().parent / "golden"


def sig(z):
    return 1.0 / (1.0 + math.exp(-z))


def rand_weights(rng, L, D, in_dim, H, scale=0.5, bias=True):
    ws = []
    for l in range(L):
        in_l = in_dim if l == 0 else D * H
        for _ in range(D):
            ws.append({
                "wx": rng.uniform(-scale, scale, (4 * H, in_l)).astype(np.float32),
                "wh": rng.uniform(-scale, scale, (4 * H, H)).astype(np.float32),
                "b": rng.uniform(-scale, scale, (4 * H,)).astype(np.float32) if bias else None,
            })
    return ws


# ---------------------------------------------------------------- closed form: all-zero matrices
def test_zero_matrices_closed_form(oracle):
    rng = np.random.default_rng(11)
    H, T, B, in_dim = 5, 9, 3, 4
    b = rng.uniform(-1.5, 1.5, 4 * H).astype(np.float32)
    ws = [{"wx": np.zeros((4 * H, in_dim), np.float32), "wh": np.zeros((4 * H, H), np.float32), "b": b}]
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-1, 1, (1, B, H))
    c0 = rng.standard_normal((1, B, H))
    y, hT, cT = oracle.forward(ws, x, h0, c0, layers=1, bidir=False, hidden=H)
    for j in range(H):
        i, f = sig(float(b[j])), sig(float(b[H + j]))
        g, o = math.tanh(float(b[2 * H + j])), sig(float(b[3 * H + j]))
        for bb in range(B):
            for t in range(1, T + 1):
                c = f ** t * c0[0, bb, j] + i * g * (1 - f ** t) / (1 - f)
                assert y[t - 1, bb, j] == pytest.approx(o * math.tanh(c), rel=1e-13, abs=1e-15)
            assert cT[0, bb, j] == pytest.approx(c, rel=1e-13, abs=1e-15)
            assert hT[0, bb, j] == y[T - 1, bb, j]


def _golden_rows(tag):
    rows = []
    for line in (GOLDEN / "hand_case_h1.txt").read_text().splitlines():
        p = line.split()
        if p and p[0] == tag:
            rows.append([float(v) for v in p[1:]])
    return rows


def test_zero_matrices_printed_instance(oracle):
    H = 1
    b = np.array([0.0, 0.0, math.atanh(0.5), 0.0], np.float64)
    # float32 storage of atanh(0.5) perturbs tanh(b_g) by < 1e-7: compare at 1e-7, and exactly
    # against the closed form evaluated with the stored float32 value.
    ws = [{"wx": np.zeros((4, 1), np.float32), "wh": np.zeros((4, 1), np.float32), "b": b.astype(np.float32)}]
    y, _, cT = oracle.forward(ws, np.ones((4, 1, 1)), layers=1, bidir=False, hidden=H)
    g32 = math.tanh(float(np.float32(b[2])))
    for t, c_gold, h_gold in _golden_rows("zero"):
        t = int(t)
        assert c_gold == 0.5 * (1 - 0.5 ** t)
        assert y[t - 1, 0, 0] == pytest.approx(h_gold, abs=1e-7)
        c = 0.5 * g32 * (1 - 0.5 ** t) / 0.5
        assert y[t - 1, 0, 0] == pytest.approx(0.5 * math.tanh(c), rel=1e-14)
    assert cT[0, 0, 0] == pytest.approx(0.46875, abs=1e-7)


# ---------------------------------------------------------------- hand-evaluated single unit
def _hand_case():
    g = {k: _golden_rows(k)[0] for k in ("wx", "wh", "b", "x")}
    return g["wx"], g["wh"], g["b"], g["x"]


def _unrolled_single_unit(wx, wh, b, xs):
    """Three steps written out one after another, no loop over time shared with the oracle."""
    wxi, wxf, wxg, wxo = wx
    whi, whf, whg, who = wh
    bi, bf, bg, bo = b
    x1, x2, x3 = xs
    c1 = sig(wxf * x1 + bf) * 0.0 + sig(wxi * x1 + bi) * math.tanh(wxg * x1 + bg)
    h1 = sig(wxo * x1 + bo) * math.tanh(c1)
    c2 = sig(wxf * x2 + whf * h1 + bf) * c1 + sig(wxi * x2 + whi * h1 + bi) * math.tanh(wxg * x2 + whg * h1 + bg)
    h2 = sig(wxo * x2 + who * h1 + bo) * math.tanh(c2)
    c3 = sig(wxf * x3 + whf * h2 + bf) * c2 + sig(wxi * x3 + whi * h2 + bi) * math.tanh(wxg * x3 + whg * h2 + bg)
    h3 = sig(wxo * x3 + who * h2 + bo) * math.tanh(c3)
    return (c1, h1), (c2, h2), (c3, h3)


def test_hand_case_golden_matches_unrolled_formula():
    wx, wh, b, xs = _hand_case()
    # the file's numbers are exact-decimal weights; evaluate in double
    fwd = _unrolled_single_unit(wx, wh, b, xs)
    for (t, c_gold, h_gold), (c, h) in zip(_golden_rows("fwd"), fwd):
        assert c == pytest.approx(c_gold, abs=2e-12) and h == pytest.approx(h_gold, abs=2e-12)
    rev = _unrolled_single_unit(wx, wh, b, xs[::-1])
    for (pos, c_gold, h_gold), (c, h) in zip(_golden_rows("rev"), rev):
        assert c == pytest.approx(c_gold, abs=2e-12) and h == pytest.approx(h_gold, abs=2e-12)
    # first step's pre-activations quoted with the case: z = (.6, -.05, .65, .15)
    z = [wx[q] * xs[0] + b[q] for q in range(4)]
    assert z == pytest.approx([0.6, -0.05, 0.65, 0.15], abs=1e-15)


def test_hand_case_oracle(oracle):
    wx, wh, b, xs = _hand_case()
    # weights chosen exactly representable or not: feed float32-rounded values to both sides
    wx32 = np.array(wx, np.float32); wh32 = np.array(wh, np.float32); b32 = np.array(b, np.float32)
    w = {"wx": wx32.reshape(4, 1), "wh": wh32.reshape(4, 1), "b": b32}
    x = np.array(xs, np.float64).reshape(3, 1, 1)
    y, hT, cT = oracle.forward([w, w], x, layers=1, bidir=True, hidden=1)
    fwd = _unrolled_single_unit(wx32.astype(float), wh32.astype(float), b32.astype(float), xs)
    rev = _unrolled_single_unit(wx32.astype(float), wh32.astype(float), b32.astype(float), xs[::-1])
    for t in range(3):
        assert y[t, 0, 0] == pytest.approx(fwd[t][1], rel=1e-14)
        assert y[2 - t, 0, 1] == pytest.approx(rev[t][1], rel=1e-14)
    assert (hT[0, 0, 0], cT[0, 0, 0]) == pytest.approx((fwd[2][1], fwd[2][0]), rel=1e-14)
    assert (hT[1, 0, 0], cT[1, 0, 0]) == pytest.approx((rev[2][1], rev[2][0]), rel=1e-14)
    # and against the file's 12-digit values (float32 storage of 0.1, 0.3, ... moves them < 1e-7)
    for (t, c_gold, h_gold) in _golden_rows("fwd"):
        assert y[int(t) - 1, 0, 0] == pytest.approx(h_gold, abs=2e-7)
    for (pos, c_gold, h_gold) in _golden_rows("rev"):
        assert y[int(pos) - 1, 0, 1] == pytest.approx(h_gold, abs=2e-7)


# ---------------------------------------------------------------- brute force, recursive definition
def brute_force(ws, x, h0, c0, L, D, H):
    """Top-down memoised evaluation of the definition: state(l,d,s,b,j) asks for what it needs."""
    T, B, in_dim = x.shape
    W = [{k: (np.asarray(v, np.float64) if v is not None else None) for k, v in w.items()} for w in ws]

    def inp(l, t, b, k):
        if l == 0:
            return float(x[t, b, k])
        d, j = divmod(k, H)
        s = t if d == 0 else T - 1 - t           # step index at which direction d produced position t
        return state(l - 1, d, s, b, j)[1]

    @lru_cache(maxsize=None)
    def state(l, d, s, b, j):
        """(c, h) of unit j after processing step index s (s = -1: initial state)."""
        if s < 0:
            return float(c0[l * D + d, b, j]), float(h0[l * D + d, b, j])
        t = s if d == 0 else T - 1 - s
        w = W[l * D + d]
        in_l = in_dim if l == 0 else D * H
        z = []
        for q in range(4):
            r = q * H + j
            acc = w["b"][r] if w["b"] is not None else 0.0
            acc += sum(w["wx"][r, k] * inp(l, t, b, k) for k in range(in_l))
            acc += sum(w["wh"][r, k] * state(l, d, s - 1, b, k)[1] for k in range(H))
            z.append(acc)
        c_prev = state(l, d, s - 1, b, j)[0]
        c = sig(z[1]) * c_prev + sig(z[0]) * math.tanh(z[2])
        return c, sig(z[3]) * math.tanh(c)

    y = np.zeros((T, B, D * H))
    hT = np.zeros((L * D, B, H)); cT = np.zeros((L * D, B, H))
    for b in range(B):
        for d in range(D):
            for j in range(H):
                for t in range(T):
                    s = t if d == 0 else T - 1 - t
                    y[t, b, d * H + j] = state(L - 1, d, s, b, j)[1]
                for l in range(L):
                    cT[l * D + d, b, j], hT[l * D + d, b, j] = state(l, d, T - 1, b, j)
    return y, hT, cT


@pytest.mark.parametrize("L,D", [(1, 1), (2, 1), (1, 2), (2, 2)])
def test_brute_force_tiny(oracle, L, D):
    rng = np.random.default_rng(100 + 10 * L + D)
    H, in_dim, T, B = 2, 3, 3, 2
    ws = rand_weights(rng, L, D, in_dim, H, scale=0.9)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
    got = oracle.forward(ws, x, h0, c0, layers=L, bidir=D == 2, hidden=H)
    ref = brute_force(ws, x, h0, c0, L, D, H)
    for g, r in zip(got, ref):
        np.testing.assert_allclose(g, r, rtol=0, atol=1e-14)


# ---------------------------------------------------------------- invariants
def test_mask_equals_explicit_zero_and_csr_walk_bitwise(oracle):
    rng = np.random.default_rng(5)
    L, D, H, in_dim, T, B = 2, 2, 7, 5, 6, 3
    ws = rand_weights(rng, L, D, in_dim, H)
    masked, zeroed, csr = [], [], []
    for l in range(L):
        for d in range(D):
            w = ws[l * D + d]
            mx = (rng.random(w["wx"].shape) < 0.3).astype(np.uint8)
            mh = (rng.random(w["wh"].shape) < 0.3).astype(np.uint8)
            mh[3] = 0                                  # an empty row: z reduces to b + Wx x
            masked.append({**w, "mask_x": mx, "mask_h": mh})
            zeroed.append({"wx": w["wx"] * mx, "wh": w["wh"] * mh, "b": w["b"]})
            csr.append({"wx_csr": oracle.dense_to_csr(w["wx"], mx),
                        "wh_csr": oracle.dense_to_csr(w["wh"], mh), "b": w["b"]})
    x = rng.standard_normal((T, B, in_dim))
    a = oracle.forward(masked, x, layers=L, bidir=True, hidden=H)
    b = oracle.forward(zeroed, x, layers=L, bidir=True, hidden=H)
    c = oracle.forward(csr, x, layers=L, bidir=True, hidden=H)
    for u, v, w_ in zip(a, b, c):
        assert np.array_equal(u, v) and np.array_equal(u, w_)
    # and the mask matters: unmasked weights give something else
    d = oracle.forward(ws, x, layers=L, bidir=True, hidden=H)
    assert np.max(np.abs(d[0] - a[0])) > 1e-3


def test_batch_columns_independent(oracle):
    rng = np.random.default_rng(6)
    L, D, H, in_dim, T, B = 2, 2, 4, 3, 5, 4
    ws = rand_weights(rng, L, D, in_dim, H)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-1, 1, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
    y, hT, cT = oracle.forward(ws, x, h0, c0, layers=L, bidir=True, hidden=H)
    for b in range(B):
        y1, h1, c1 = oracle.forward(ws, x[:, b:b + 1], h0[:, b:b + 1], c0[:, b:b + 1], layers=L, bidir=True, hidden=H)
        assert np.array_equal(y1[:, 0], y[:, b]) and np.array_equal(h1[:, 0], hT[:, b]) and np.array_equal(c1[:, 0], cT[:, b])


def test_reverse_is_forward_on_reversed_time(oracle):
    rng = np.random.default_rng(7)
    H, in_dim, T, B = 5, 4, 7, 2
    ws = rand_weights(rng, 1, 2, in_dim, H)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-1, 1, (2, B, H)); c0 = rng.standard_normal((2, B, H))
    y, hT, cT = oracle.forward(ws, x, h0, c0, layers=1, bidir=True, hidden=H)
    yf, hf, cf = oracle.forward([ws[0]], x, h0[:1], c0[:1], layers=1, bidir=False, hidden=H)
    yr, hr, cr = oracle.forward([ws[1]], x[::-1], h0[1:], c0[1:], layers=1, bidir=False, hidden=H)
    assert np.array_equal(y[:, :, :H], yf) and np.array_equal(y[:, :, H:], yr[::-1])
    assert np.array_equal(hT[0], hf[0]) and np.array_equal(hT[1], hr[0]) and np.array_equal(cT[1], cr[0])


def test_stack_is_composition_and_chunking_carries_state(oracle):
    rng = np.random.default_rng(8)
    L, H, in_dim, T, B = 3, 4, 6, 9, 2
    ws = rand_weights(rng, L, 1, in_dim, H)
    x = rng.standard_normal((T, B, in_dim))
    y, hT, cT = oracle.forward(ws, x, layers=L, bidir=False, hidden=H)
    cur = x
    for l in range(L):
        cur, h1, c1 = oracle.forward([ws[l]], cur, layers=1, bidir=False, hidden=H)
        assert np.array_equal(h1[0], hT[l]) and np.array_equal(c1[0], cT[l])
    assert np.array_equal(cur, y)
    ya, ha, ca = oracle.forward(ws, x[:5], layers=L, bidir=False, hidden=H)
    yb, hb, cb = oracle.forward(ws, x[5:], ha, ca, layers=L, bidir=False, hidden=H)
    assert np.array_equal(np.concatenate([ya, yb]), y) and np.array_equal(hb, hT) and np.array_equal(cb, cT)


def test_gate_roles_are_distinct_and_bounds_hold(oracle):
    """Swapping two gate blocks of (W, b) changes the output (so a swapped block cannot hide), and
    |h| < 1, |c_t| <= |c_{t-1}| + 1."""
    rng = np.random.default_rng(9)
    H, in_dim, T, B = 6, 5, 8, 2
    ws = rand_weights(rng, 1, 1, in_dim, H, scale=1.0)
    x = rng.standard_normal((T, B, in_dim))
    y, hT, cT = oracle.forward(ws, x, layers=1, bidir=False, hidden=H)
    assert np.all(np.abs(y) < 1) and np.all(np.abs(cT) <= T)
    for a, b in [(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)]:
        perm = list(range(4)); perm[a], perm[b] = perm[b], perm[a]
        idx = np.concatenate([np.arange(q * H, (q + 1) * H) for q in perm])
        w2 = [{"wx": ws[0]["wx"][idx], "wh": ws[0]["wh"][idx], "b": ws[0]["b"][idx]}]
        y2, _, _ = oracle.forward(w2, x, layers=1, bidir=False, hidden=H)
        assert np.max(np.abs(y2 - y)) > 1e-3, (a, b)


def test_hidden_unit_relabelling(oracle):
    """Permuting hidden units (rows of every gate block, columns of Wh, the state) permutes y."""
    rng = np.random.default_rng(10)
    H, in_dim, T, B = 6, 3, 5, 2
    ws = rand_weights(rng, 1, 1, in_dim, H)
    x = rng.standard_normal((T, B, in_dim))
    p = rng.permutation(H)
    rows = np.concatenate([q * H + p for q in range(4)])
    w2 = [{"wx": ws[0]["wx"][rows], "wh": ws[0]["wh"][rows][:, p], "b": ws[0]["b"][rows]}]
    y, _, _ = oracle.forward(ws, x, layers=1, bidir=False, hidden=H)
    y2, _, _ = oracle.forward(w2, x, layers=1, bidir=False, hidden=H)
    np.testing.assert_allclose(y2, y[:, :, p], rtol=0, atol=1e-15)   # summation order over k changes


# ---------------------------------------------------------------- library special case
def torch_lstm_reference(ws, x, h0, c0, L, D, H):
    import torch
    T, B, in_dim = x.shape
    m = torch.nn.LSTM(in_dim, H, num_layers=L, bidirectional=(D == 2)).double()
    with torch.no_grad():
        for l in range(L):
            for d in range(D):
                sfx = f"_l{l}" + ("_reverse" if d else "")
                w = ws[l * D + d]
                wx = np.asarray(w["wx"], np.float64); wh = np.asarray(w["wh"], np.float64)
                if w.get("mask_x") is not None:
                    wx = wx * w["mask_x"]; wh = wh * w["mask_h"]
                getattr(m, "weight_ih" + sfx).copy_(torch.from_numpy(wx))
                getattr(m, "weight_hh" + sfx).copy_(torch.from_numpy(wh))
                getattr(m, "bias_ih" + sfx).copy_(torch.from_numpy(np.asarray(w["b"], np.float64)))
                getattr(m, "bias_hh" + sfx).zero_()
        z = torch.zeros(L * D, B, H, dtype=torch.float64)
        hh = torch.from_numpy(np.asarray(h0, np.float64)) if h0 is not None else z
        cc = torch.from_numpy(np.asarray(c0, np.float64)) if c0 is not None else z
        y, (hT, cT) = m(torch.from_numpy(np.asarray(x, np.float64)), (hh, cc))
    return y.numpy(), hT.numpy(), cT.numpy()


SCALED = [
    wl.config1().with_(T=12, B=5),
    wl.config2(1).with_(in_dim=96, hidden=72, T=11, B=3),
    wl.config3(136).with_(T=9),
    wl.config4(0.10).with_(in_dim=120, hidden=88, T=10, B=2),
    wl.config5(1).with_(layers=3, in_dim=50, hidden=40, T=14, B=3),
]


@pytest.mark.parametrize("w", SCALED, ids=lambda w: w.name)
def test_against_torch_float64_lstm_scaled_shapes(oracle, w):
    ws, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    got = oracle.forward(ws, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    ref = torch_lstm_reference(ws, x, h0, c0, w.layers, w.dirs, w.hidden)
    for g, r in zip(got, ref):
        np.testing.assert_allclose(g, r, rtol=0, atol=1e-12)


def test_against_torch_float64_lstm_config1_full(oracle):
    w = wl.config1()
    ws, x = wl.make(w)
    got = oracle.forward(ws, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    ref = torch_lstm_reference(ws, x, None, None, w.layers, w.dirs, w.hidden)
    for g, r in zip(got, ref):
        np.testing.assert_allclose(g, r, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- planted mistakes are caught
MUTATIONS = {
    "forget/input swapped": ("double gi = sigma(z[0]);\n                double gf = sigma(z[1]);",
                             "double gi = sigma(z[1]);\n                double gf = sigma(z[0]);"),
    "cell gate uses sigmoid": ("double gg = tanh(z[2]);", "double gg = sigma(z[2]);"),
    "output gate row wrong": ("double go = sigma(z[3]);", "double go = sigma(z[2]);"),
    "bias dropped": ("double acc = w->b ? (double)w->b[row] : 0.0;", "double acc = 0.0;"),
    "sigmoid sign": ("return 1.0 / (1.0 + exp(-z));", "return 1.0 / (1.0 + exp(z));"),
    "cell update drops carry": ("double c = gf * c_prev[(size_t)b * H + j] + gi * gg;", "double c = gi * gg;"),
    "h without tanh": ("double h = go * tanh(c);", "double h = go * c;"),
    "reverse ignored": ("int t = reverse ? T - 1 - s : s;", "int t = s;"),
    "state index": ("size_t s = (size_t)(l * D + d) * st_n;", "size_t s = (size_t)(l + d) * st_n;"),
    "concat offset": ("Y, D * H, d * H,", "Y, D * H, 0,"),
    "recurrent term dropped": ("acc = add_row_product(acc, row, H, w->wh,", "if (0) acc = add_row_product(acc, row, H, w->wh,"),
    "gate row stride": ("int row = q * H + j;", "int row = j * 4 + q;"),
}
MUTATIONS["adjacent weights swapped in dense walk"] = (
    "double w = (double)r[k];", "double w = (double)dense[((size_t)row * ncol + k) ^ 1];")
MUTATIONS["wrong row in dense walk"] = (
    "const float *r = dense + (size_t)row * ncol;", "const float *r = dense + (size_t)(row % ncol) * ncol;")


def _run_pins_on(lib_path):
    """Re-run the tiny brute-force pin (all four L x D shapes) on an alternative oracle build."""
    lib = ctypes.CDLL(str(lib_path))
    lib.lstm_oracle_forward.restype = ctypes.c_int
    lib.lstm_oracle_forward.argtypes = [ctypes.c_int] * 6 + [ctypes.c_void_p] * 7
    import oracle.lstm_oracle as lo
    saved = lo._lib
    lo._lib = lib
    try:
        worst = 0.0
        for L, D in [(1, 1), (2, 2)]:
            rng = np.random.default_rng(100 + 10 * L + D)
            H, in_dim, T, B = 2, 3, 3, 2
            ws = rand_weights(rng, L, D, in_dim, H, scale=0.9)
            x = rng.standard_normal((T, B, in_dim))
            h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
            got = lo.forward(ws, x, h0, c0, layers=L, bidir=D == 2, hidden=H)
            ref = brute_force(ws, x, h0, c0, L, D, H)
            worst = max(worst, max(float(np.max(np.abs(g - r))) for g, r in zip(got, ref)))
        return worst
    finally:
        lo._lib = saved


@pytest.mark.skipif(shutil.which("gcc") is None, reason="gcc needed")
def test_planted_mistakes_are_caught(oracle, tmp_path):
    src = (Path(oracle.__file__).resolve().parent / "lstm_oracle.c").read_text()

    def compile_variant(text, name):
        c = tmp_path / f"{name}.c"; so = tmp_path / f"{name}.so"
        c.write_text(text)
        subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(so), str(c), "-lm"], check=True)
        return so

    assert _run_pins_on(compile_variant(src, "clean")) < 1e-14
    for n, (name, (old, new)) in enumerate(MUTATIONS.items()):
        assert src.count(old) >= 1, f"mutation target not found: {name}"
        worst = _run_pins_on(compile_variant(src.replace(old, new, 1), f"mut{n}"))
        assert worst > 1e-6, f"planted mistake not caught: {name}"


# ---------------------------------------------------------------- the projection on its own
def test_input_projection_definition_and_its_tie_to_the_cell(oracle):
    """oracle.input_projection is the matrix product written out; it is pinned by explicit loops on a tiny
    case and by the cell oracle: with Wh = 0 and zero initial state, one step gives
    h = sigmoid(g_o) tanh(sigmoid(g_i) tanh(g_g)) from the projection values alone."""
    rng = np.random.default_rng(77)
    H, in_dim, T, B = 3, 4, 2, 2
    ws = rand_weights(rng, 1, 2, in_dim, H, scale=0.8)
    mask = (rng.random((4 * H, in_dim)) < 0.6).astype(np.uint8)
    ws[1]["mask_x"] = mask
    x = rng.standard_normal((T, B, in_dim))
    g = oracle.input_projection(ws, x, bidir=True, hidden=H)
    for d in range(2):
        for t in range(T):
            for b in range(B):
                for r in range(4 * H):
                    acc = float(ws[d]["b"][r])
                    for k in range(in_dim):
                        keep = 1.0 if (d == 0 or mask[r, k]) else 0.0
                        acc += float(ws[d]["wx"][r, k]) * keep * x[t, b, k]
                    assert g[t, b, d, r] == pytest.approx(acc, rel=1e-13, abs=1e-15)
    # tie to the cell: first step of the forward direction, no recurrent weights
    w0 = {**ws[0], "wh": np.zeros((4 * H, H), np.float32)}
    y, _, _ = oracle.forward([w0], x[:1], layers=1, bidir=False, hidden=H)
    for b in range(B):
        for j in range(H):
            gi, gg, go = g[0, b, 0, j], g[0, b, 0, 2 * H + j], g[0, b, 0, 3 * H + j]
            assert y[0, b, j] == pytest.approx(sig(go) * math.tanh(sig(gi) * math.tanh(gg)), rel=1e-13)
    # CSR description of the same matrix
    csr = [{"wx_csr": oracle.dense_to_csr(ws[1]["wx"], mask), "b": ws[1]["b"]}]
    g_csr = oracle.input_projection(csr, x, bidir=False, hidden=H)
    assert np.array_equal(g_csr[:, :, 0], g[:, :, 1])
