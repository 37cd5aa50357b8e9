"""The code paths the environment switches select instead of the defaults must stay correct: they are what the
defaults are measured against (issuing threads of the batched recurrence, 128-row projection tiles, the
list-walking projection of CSR handles), and some are the only path for shapes the default does not serve."""
import numpy as np
import pytest

import lstm_workloads as wl
from gpu_util import assert_close, csr_weights

pytestmark = pytest.mark.gpu


def small(name, layers, bidir, in_dim, hidden, T, B, dtype, scale=0.1, seed=7, density=1.0):
    return wl.Workload(name, layers, bidir, in_dim, hidden, T, B, dtype, scale, density=density, seed=seed)


def _forward(pkg, w, weights, x, h0, c0, exec_mode="dense"):
    import torch
    m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype=w.dtype,
                 exec_mode=exec_mode, max_T=w.T, max_B=w.B)
    try:
        y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
        m.check()
        return (y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), m.info()
    finally:
        m.close()


@pytest.mark.parametrize("issuers", ["1", "2"])
def test_batched_recurrence_with_fewer_issuing_threads(oracle, issuers, monkeypatch):
    """One and two issuing threads (one and two accumulators) instead of three; pair mode and both directions,
    and a slice whose ring does not hold a whole step's operand."""
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_TC_ISSUE", issuers)
    for w in (small("tci_h600_b20", 1, True, 24, 600, 3, 20, "bf16", scale=0.05),
              small("tci_h1600_b9", 1, False, 32, 1600, 2, 9, "bf16", scale=0.03)):
        weights, x = wl.make(w)
        h0, c0 = wl.make_states(w)
        ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
        got, info = _forward(pkg, w, weights, x, h0, c0)
        assert info["recur_batched_tensor_core"] >= 1
        assert_close(got, ref, "bf16", f"{w.name}/issuers={issuers}")


def test_batched_recurrence_without_cluster_pairs(oracle, monkeypatch):
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_RECUR", "tc1")
    w = small("tc1_h600_b20", 2, False, 24, 600, 3, 20, "bf16", scale=0.05)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got, info = _forward(pkg, w, weights, x, h0, c0)
    assert info["recur_batched_tensor_core"] == 1
    assert_close(got, ref, "bf16", w.name)


@pytest.mark.parametrize("tile", ["128", ""])
def test_projection_tiles_at_several_activation_tiles(oracle, tile, monkeypatch):
    """T*B = 390 rows (four activation tiles, a ragged last one) and 4H = 1160 weight rows (a ragged 256-row tile):
    the persistent 256-row kernel (default) and the 128-row kernel, through the whole forward pass."""
    import paper_1901_10997_b200 as pkg
    if tile:
        monkeypatch.setenv("LSTM_B200_PROJ_TILE", tile)
    else:
        monkeypatch.delenv("LSTM_B200_PROJ_TILE", raising=False)
    w = small("proj_tiles", 2, False, 200, 290, 13, 30, "bf16", scale=0.05)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got, _ = _forward(pkg, w, weights, x, h0, c0)
    assert_close(got, ref, "bf16", f"{w.name}/tile={tile or 'default'}")


@pytest.mark.parametrize("proj", ["csr", ""])
def test_csr_handle_with_either_projection(oracle, proj, monkeypatch):
    """bf16 CSR handles project on the tensor cores over a dense copy of Wx by default and walk the lists with
    LSTM_B200_PROJ=csr; two layers, so that the second projection reads what the sparse recurrence wrote."""
    import paper_1901_10997_b200 as pkg
    if proj:
        monkeypatch.setenv("LSTM_B200_PROJ", proj)
    else:
        monkeypatch.delenv("LSTM_B200_PROJ", raising=False)
    for B in (1, 3):
        w = small("csr_proj", 2, True, 70, 200, 6, B, "bf16", scale=0.2, density=0.15, seed=5)
        weights, x = wl.make(w)
        h0, c0 = wl.make_states(w)
        ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
        got, info = _forward(pkg, w, csr_weights(oracle, weights), x, h0, c0, exec_mode="csr")
        assert info["proj_tensor_core"] == (0 if proj else 1)
        assert_close(got, ref, "bf16", f"{w.name}/B={B}/proj={proj or 'default'}")


@pytest.mark.parametrize("T,fused", [(37, True), (41, False)])
def test_sparse_kernel_projects_in_its_prologue_for_short_single_sequences(oracle, T, fused, monkeypatch):
    """bf16 CSR handle on the 16-warp register-resident sparse kernel (H > 512): one sequence of at most 40 steps
    computes its projection inside the recurrent launch (two launches for two layers), a longer one does not;
    both directions, a ragged last timestep tile, non-zero initial state."""
    import torch
    import paper_1901_10997_b200 as pkg
    monkeypatch.delenv("LSTM_B200_PROJ", raising=False)
    monkeypatch.delenv("LSTM_B200_FUSE", raising=False)
    w = small("csr_fused", 2, True, 90, 600, T, 1, "bf16", scale=0.15, density=0.1, seed=9)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    m = pkg.LSTM(csr_weights(oracle, weights), layers=2, in_dim=w.in_dim, hidden=w.hidden, bidir=True, dtype="bf16",
                 exec_mode="csr", max_T=T, max_B=1)
    try:
        assert m.info()["recur_csr_register_resident"] == 1
        y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
        m.check()
        assert m.info()["launches_per_forward"] == (2 if fused else 5)
        assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"{w.name}/T={T}")
    finally:
        m.close()


def _random_cases(n, seed):
    """Shapes nobody picked by hand for the paths added last: sparse and dense single sequences around the 40-step
    limit of the fused prologue, and batches whose T*B spans several activation tiles of the projection."""
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        kind = ["csr1", "dense1", "projbig"][i % 3]
        L, bidir = int(rng.integers(1, 3)), bool(rng.integers(0, 2))
        if kind == "csr1":
            c = dict(H=int(rng.integers(520, 1500)), B=int(rng.integers(1, 4)), T=int(rng.integers(1, 45)), in_dim=int(rng.integers(1, 300)),
                     mode="csr", density=float(rng.choice([0.05, 0.1, 0.3])))
        elif kind == "dense1":
            c = dict(H=int(rng.integers(100, 1600)), B=1, T=int(rng.integers(1, 45)), in_dim=int(rng.integers(1, 400)), mode="dense", density=1.0)
        else:
            c = dict(H=int(rng.integers(30, 500)), B=int(rng.integers(8, 40)), T=int(rng.integers(6, 30)), in_dim=int(rng.integers(8, 300)),
                     mode="dense", density=1.0)
        cases.append(dict(c, kind=kind, L=L, bidir=bidir, seed=7000 + i))
    return cases


@pytest.mark.parametrize("c", _random_cases(24, 31), ids=lambda c: "{kind}_L{L}D{d}_in{in_dim}_H{H}_T{T}_B{B}".format(d=1 + c["bidir"], **c))
def test_random_shapes_of_the_fused_and_large_projection_paths(oracle, c):
    import paper_1901_10997_b200 as pkg
    scale = min(0.3, 2.0 / np.sqrt(c["H"] + c["in_dim"]))
    w = wl.Workload("rnd", c["L"], c["bidir"], c["in_dim"], c["H"], c["T"], c["B"], "bf16", scale, density=c["density"], seed=c["seed"])
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got, _ = _forward(pkg, w, weights if c["mode"] == "dense" else csr_weights(oracle, weights), x, h0, c0, exec_mode=c["mode"])
    assert_close(got, ref, "bf16", "rnd/" + c["kind"])
