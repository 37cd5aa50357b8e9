"""Pins of the H-LSTM oracle (one ReLU hidden layer inside each gate; paper Section 4, the cell-equation
block with H* = one hidden layer) against things other than itself (CPU only).

The paper prints no worked example of the H-LSTM cell, so the pins are: the closed form when the hidden
layers see nothing (all-zero U) or are switched off (ReLU input pushed far below zero); the reduction to
the plain LSTM oracle -- itself pinned in test_oracle_pins.py -- when every gate's output matrix is the
identity (or a permutation) and the ReLU is held in its linear range; a brute-force recursive evaluation
on tiny stacks; a step-by-step composition from library primitives (float64 linear maps of PyTorch on
CPU); and planted mistakes that the pins must catch.
"""
import ctypes
import math
import shutil
import subprocess
from pathlib import Path

import numpy as np
import pytest


def sig(z):
    return 1.0 / (1.0 + math.exp(-z))


def rand_hweights(rng, L, D, in_dim, H, Hh, scale=0.6):
    ws = []
    for l in range(L):
        in_l = in_dim if l == 0 else D * H
        for _ in range(D):
            ws.append({
                "ux": rng.uniform(-scale, scale, (4 * Hh, in_l)).astype(np.float32),
                "uh": rng.uniform(-scale, scale, (4 * Hh, H)).astype(np.float32),
                "a": rng.uniform(-scale, scale, (4 * Hh,)).astype(np.float32),
                "w": rng.uniform(-scale, scale, (4 * H, Hh)).astype(np.float32),
                "b": rng.uniform(-scale, scale, (4 * H,)).astype(np.float32),
            })
    return ws


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("mode", ["zero_U", "relu_off"])
def test_constant_gates_closed_form(oracle, mode):
    """With U = 0 the hidden layers are relu(a); with a far below zero they are 0.  Either way the gate
    pre-activations are constants z = b + W relu(.), and c_t = f^t c_0 + i g (1 - f^t) / (1 - f)."""
    rng = np.random.default_rng(3)
    H, Hh, T, B, in_dim = 4, 6, 7, 2, 3
    w = rand_hweights(rng, 1, 1, in_dim, H, Hh)[0]
    if mode == "zero_U":
        w["ux"][:] = 0; w["uh"][:] = 0
        r = np.maximum(w["a"].astype(np.float64), 0.0)
    else:
        w["a"][:] = -1e4
        r = np.zeros(4 * Hh)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-1, 1, (1, B, H)); c0 = rng.standard_normal((1, B, H))
    y, hT, cT = oracle.forward_hlstm([w], x, h0, c0, layers=1, bidir=False, hidden=H, gate_hidden=Hh)
    z = np.array([[float(w["b"][q * H + j]) + float(np.dot(w["w"][q * H + j].astype(np.float64), r[q * Hh:(q + 1) * Hh]))
                   for j in range(H)] for q in range(4)])
    for j in range(H):
        i, f, g, o = sig(z[0, j]), sig(z[1, j]), math.tanh(z[2, j]), sig(z[3, j])
        for b in range(B):
            for t in range(1, T + 1):
                c = f ** t * c0[0, b, j] + i * g * (1 - f ** t) / (1 - f)
                assert y[t - 1, b, j] == pytest.approx(o * math.tanh(c), rel=1e-12, abs=1e-14)
            assert cT[0, b, j] == pytest.approx(c, rel=1e-12, abs=1e-14)


# ---------------------------------------------------------------- reduction to the plain LSTM
@pytest.mark.parametrize("L,D", [(1, 1), (2, 2)])
@pytest.mark.parametrize("permute", [False, True])
def test_identity_output_matrices_reduce_to_the_lstm_oracle(oracle, L, D, permute):
    """Hh = H, W_q = a permutation P_q (or I), and the hidden bias shifted by S so that the ReLU never
    clips: z_q = b_q + P_q (a_q + S + Ux_q x + Uh_q h).  Taking b_q = b0_q - S this is the plain LSTM with
    Wx = P_q Ux_q, Wh = P_q Uh_q and bias b0_q + P_q a_q."""
    rng = np.random.default_rng(10 * L + D + (5 if permute else 0))
    H = Hh = 5
    in_dim, T, B, S = 3, 6, 2, 64.0
    hws, lws = [], []
    for l in range(L):
        in_l = in_dim if l == 0 else D * H
        for _ in range(D):
            ux = rng.uniform(-0.7, 0.7, (4 * Hh, in_l)).astype(np.float32)
            uh = rng.uniform(-0.7, 0.7, (4 * Hh, H)).astype(np.float32)
            a0 = rng.uniform(-0.5, 0.5, 4 * Hh).astype(np.float32)
            b0 = rng.uniform(-0.5, 0.5, 4 * H).astype(np.float32)
            w = np.zeros((4 * H, Hh), np.float32)
            wx = np.zeros_like(ux); wh = np.zeros_like(uh); bias = np.zeros(4 * H, np.float32)
            for q in range(4):
                perm = rng.permutation(H) if permute else np.arange(H)
                for j in range(H):
                    w[q * H + j, perm[j]] = 1.0
                    wx[q * H + j] = ux[q * Hh + perm[j]]
                    wh[q * H + j] = uh[q * Hh + perm[j]]
                    bias[q * H + j] = np.float32(b0[q * H + j] + a0[q * Hh + perm[j]])
            hws.append({"ux": ux, "uh": uh, "a": (a0 + np.float32(S)).astype(np.float32), "w": w,
                        "b": (b0 - np.float32(S)).astype(np.float32)})
            lws.append({"wx": wx, "wh": wh, "b": bias})
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
    got = oracle.forward_hlstm(hws, x, h0, c0, layers=L, bidir=D == 2, hidden=H, gate_hidden=Hh)
    ref = oracle.forward(lws, x, h0, c0, layers=L, bidir=D == 2, hidden=H)
    for g, r in zip(got, ref):
        # float32 storage of a0 + S, b0 - S and of the folded bias moves z by at most a few 1e-6
        assert np.max(np.abs(g - r)) < 2e-5


# ---------------------------------------------------------------- brute force on tiny stacks
def brute_force(ws, x, h0, c0, L, D, H, Hh):
    """Recursive per-output evaluation, written separately from the oracle's loops."""
    T, B, in_dim = x.shape
    memo = {}

    def inp(l, t, b, k):
        if l == 0:
            return float(x[t, b, k])
        d, j = divmod(k, H)
        return state(l - 1, d, t, b, j)[1]

    def state(l, d, t, b, j):
        """(c, h) of layer l, direction d after processing position t."""
        key = (l, d, t, b, j)
        if key in memo:
            return memo[key]
        w = ws[l * D + d]
        in_l = in_dim if l == 0 else D * H
        prev_t = t + 1 if d == 1 else t - 1
        first = (t == T - 1) if d == 1 else (t == 0)

        def hprev(k):
            return float(h0[l * D + d, b, k]) if first else state(l, d, prev_t, b, k)[1]

        cprev = float(c0[l * D + d, b, j]) if first else state(l, d, prev_t, b, j)[0]
        z = []
        for q in range(4):
            acc = float(w["b"][q * H + j])
            for m in range(Hh):
                pre = float(w["a"][q * Hh + m])
                pre += sum(float(w["ux"][q * Hh + m, k]) * inp(l, t, b, k) for k in range(in_l))
                pre += sum(float(w["uh"][q * Hh + m, k]) * hprev(k) for k in range(H))
                acc += float(w["w"][q * H + j, m]) * max(pre, 0.0)
            z.append(acc)
        c = sig(z[1]) * cprev + sig(z[0]) * math.tanh(z[2])
        h = sig(z[3]) * math.tanh(c)
        memo[key] = (c, h)
        return memo[key]

    y = np.zeros((T, B, D * H)); hT = np.zeros((L * D, B, H)); cT = np.zeros((L * D, B, H))
    for d in range(D):
        for b in range(B):
            for j in range(H):
                for t in range(T):
                    y[t, b, d * H + j] = state(L - 1, d, t, b, j)[1]
                for l in range(L):
                    cT[l * D + d, b, j], hT[l * D + d, b, j] = state(l, d, 0 if d == 1 else T - 1, b, j)
    return y, hT, cT


@pytest.mark.parametrize("L,D", [(1, 1), (2, 1), (1, 2), (2, 2)])
def test_brute_force_tiny(oracle, L, D):
    rng = np.random.default_rng(40 + 10 * L + D)
    H, Hh, in_dim, T, B = 2, 3, 3, 3, 2
    ws = rand_hweights(rng, L, D, in_dim, H, Hh, scale=0.9)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
    got = oracle.forward_hlstm(ws, x, h0, c0, layers=L, bidir=D == 2, hidden=H, gate_hidden=Hh)
    ref = brute_force(ws, x, h0, c0, L, D, H, Hh)
    for g, r in zip(got, ref):
        assert np.max(np.abs(g - r)) < 1e-14


# ---------------------------------------------------------------- composition from library primitives
def torch_composition(ws, x, h0, c0, L, D, H, Hh):
    import torch
    import torch.nn.functional as F
    X = torch.from_numpy(np.asarray(x, np.float64))
    T, B, _ = X.shape
    hT = torch.zeros((L * D, B, H), dtype=torch.float64); cT = torch.zeros_like(hT)
    for l in range(L):
        outs = []
        for d in range(D):
            w = {k: torch.from_numpy(np.asarray(v, np.float64)) for k, v in ws[l * D + d].items()}
            h = torch.from_numpy(np.asarray(h0[l * D + d], np.float64)); c = torch.from_numpy(np.asarray(c0[l * D + d], np.float64))
            ys = [None] * T
            for t in (range(T - 1, -1, -1) if d == 1 else range(T)):
                r = F.relu(F.linear(X[t], w["ux"]) + F.linear(h, w["uh"]) + w["a"])          # [B, 4Hh]
                z = torch.stack([F.linear(r[:, q * Hh:(q + 1) * Hh], w["w"][q * H:(q + 1) * H]) + w["b"][q * H:(q + 1) * H]
                                 for q in range(4)])
                c = torch.sigmoid(z[1]) * c + torch.sigmoid(z[0]) * torch.tanh(z[2])
                h = torch.sigmoid(z[3]) * torch.tanh(c)
                ys[t] = h
            outs.append(torch.stack(ys))
            hT[l * D + d], cT[l * D + d] = h, c
        X = torch.cat(outs, dim=2)
    return X.numpy(), hT.numpy(), cT.numpy()


@pytest.mark.parametrize("shape", [(1, 1, 40, 33, 21, 9, 3), (2, 2, 17, 24, 24, 6, 2), (3, 1, 8, 16, 40, 5, 4)])
def test_against_float64_composition_of_linear_maps(oracle, shape):
    L, D, in_dim, H, Hh, T, B = shape
    rng = np.random.default_rng(sum(shape))
    ws = rand_hweights(rng, L, D, in_dim, H, Hh, scale=0.3)
    x = rng.standard_normal((T, B, in_dim))
    h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
    got = oracle.forward_hlstm(ws, x, h0, c0, layers=L, bidir=D == 2, hidden=H, gate_hidden=Hh)
    ref = torch_composition(ws, x, h0, c0, L, D, H, Hh)
    for g, r in zip(got, ref):
        assert np.max(np.abs(g - r)) < 1e-12


# ---------------------------------------------------------------- planted mistakes
MUTATIONS = {
    "relu dropped": ("r[(size_t)b * 4 * Hh + m] = acc > 0.0 ? acc : 0.0;", "r[(size_t)b * 4 * Hh + m] = acc;"),
    "hidden bias dropped": ("double acc = w->a ? (double)w->a[m] : 0.0;", "double acc = 0.0;"),
    "recurrent half of U dropped": ("for (int k = 0; k < H; ++k) acc += (double)w->uh[(size_t)m * H + k] * h_p[k];", ";"),
    "input half of U transposed stride": ("(double)w->ux[(size_t)m * in_l + k] * x_t[k]", "(double)w->ux[((size_t)m * in_l + k) ^ 1] * x_t[k]"),
    "every gate reads the first hidden block": ("const double *rq = r + (size_t)b * 4 * Hh + (size_t)q * Hh;", "const double *rq = r + (size_t)b * 4 * Hh;"),
    "output matrix row stride": ("acc += (double)w->w[(size_t)row * Hh + m] * rq[m];", "acc += (double)w->w[(size_t)row * H + m] * rq[m];"),
    "output bias dropped": ("double acc = w->b ? (double)w->b[row] : 0.0;\n                    for (int m = 0; m < Hh; ++m)", "double acc = 0.0;\n                    for (int m = 0; m < Hh; ++m)"),
}


def _worst_error_of(lib_path):
    lib = ctypes.CDLL(str(lib_path))
    lib.hlstm_oracle_forward.restype = ctypes.c_int
    lib.hlstm_oracle_forward.argtypes = [ctypes.c_int] * 7 + [ctypes.c_void_p] * 7
    import oracle.lstm_oracle as lo
    saved = lo._lib
    lo._lib = lib
    try:
        worst = 0.0
        for L, D in [(1, 1), (2, 2)]:
            rng = np.random.default_rng(200 + 10 * L + D)
            H, Hh, in_dim, T, B = 2, 3, 3, 3, 2
            ws = rand_hweights(rng, L, D, in_dim, H, Hh, scale=0.9)
            x = rng.standard_normal((T, B, in_dim))
            h0 = rng.uniform(-0.9, 0.9, (L * D, B, H)); c0 = rng.standard_normal((L * D, B, H))
            got = lo.forward_hlstm(ws, x, h0, c0, layers=L, bidir=D == 2, hidden=H, gate_hidden=Hh)
            ref = brute_force(ws, x, h0, c0, L, D, H, Hh)
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

    assert _worst_error_of(compile_variant(src, "clean")) < 1e-14
    for n, (name, (old, new)) in enumerate(MUTATIONS.items()):
        assert src.count(old) == 1, f"mutation target not found exactly once: {name}"
        worst = _worst_error_of(compile_variant(src.replace(old, new, 1), f"mut{n}"))
        assert worst > 1e-6, f"planted mistake not caught: {name}"
