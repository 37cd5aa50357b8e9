"""Row/column-pruned stacks on the GPU: the library runs them on the surviving units only and must return what
the oracle returns for the full model with the zeros left in (paper, Section 4.2, Algorithm 1; Table 1 step (b):
hidden width 1500 pruned to 1197)."""
import numpy as np
import pytest

import lstm_workloads as wl
from gpu_util import assert_close, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _always_compact(monkeypatch):
    """Handles for a few sequences keep the zeros by default (the narrower model is not faster there); these
    tests are about the compacted path, so it is switched on for every batch size."""
    monkeypatch.setenv("LSTM_B200_COMPACT", "1")


def _run(w, weights, x, h0, c0, exec_mode="dense", expect_hc=None):
    import torch
    import paper_1901_10997_b200 as pkg
    m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype=w.dtype,
                 exec_mode=exec_mode, max_T=w.T, max_B=w.B)
    try:
        info = m.info()
        if expect_hc is not None:
            assert info["compact_hidden"] == expect_hc, info
        dev = torch.device("cuda:0")
        t = lambda a: None if a is None else torch.from_numpy(a).to(dev)
        y, hT, cT = m.forward(t(x), t(h0), t(c0))
        m.check()
        return (y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), info
    finally:
        m.close()


@pytest.mark.parametrize("case", [("fp32", 2, True, 9, 40, 29, 5, 3, "dense"), ("bf16", 3, False, 33, 150, 101, 6, 2, "dense"),
                                  ("bf16", 2, True, 20, 96, 64, 4, 7, "dense"), ("bf16", 2, False, 16, 120, 80, 5, 1, "csr")],
                         ids=lambda c: f"{c[0]}_L{c[1]}D{1 + c[2]}_H{c[4]}to{c[5]}_B{c[7]}_{c[8]}")
def test_pruned_units_small(oracle, case):
    dtype, L, bidir, in_dim, H, keep, T, B, mode = case
    w = wl.Workload("rc_small", L, bidir, in_dim, H, T, B, dtype, 0.3, seed=900 + H)
    weights, x = wl.make(w)
    pruned, _removed = wl.prune_units(w, weights, keep)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(pruned, x, h0, c0, layers=L, bidir=bidir, hidden=H)
    got, info = _run(w, pruned, x, h0, c0, exec_mode=mode, expect_hc=keep)
    assert info["units_removed"] == L * (2 if bidir else 1) * (H - keep)
    assert_close(got, ref, dtype, "units pruned " + mode)


def test_matrices_with_different_numbers_of_pruned_units_share_one_width(oracle):
    """Layer 0 loses 30 units, layer 1 only 10: the common width is that of the fuller layer and layer 0 keeps
    twenty removable units (harmless: their rows are zero)."""
    w = wl.Workload("rc_uneven", 2, False, 24, 100, 5, 2, "bf16", 0.3, seed=31)
    weights, x = wl.make(w)
    p0, r0 = wl.prune_units(w.with_(layers=1), weights[:1], 70)
    p1, r1 = wl.prune_units(w.with_(layers=1, in_dim=100), weights[1:], 90, seed_offset=12)
    pruned = [p0[0], p1[0]]
    pruned[1]["wx"][:, r0[0]] = 0.0                     # layer 0's removed units feed nobody
    ref = oracle.forward(pruned, x, layers=2, bidir=False, hidden=100)
    got, info = _run(w, pruned, x, None, None, expect_hc=90)
    assert info["units_removed"] == 10 + 10
    assert_close(got, ref, "bf16", "uneven")


def test_unit_with_zero_rows_that_is_still_read_stays(oracle):
    w = wl.Workload("rc_read", 1, False, 12, 64, 5, 2, "bf16", 0.3, seed=32)
    weights, x = wl.make(w)
    rows = np.arange(4) * 64 + 7
    weights[0]["wx"][rows] = 0.0
    weights[0]["wh"][rows] = 0.0
    ref = oracle.forward(weights, x, layers=1, bidir=False, hidden=64)
    got, info = _run(w, weights, x, None, None, expect_hc=0)
    assert_close(got, ref, "bf16", "still read")


@pytest.mark.parametrize("B", [1, 20])
def test_config2_units_pruned_1500_to_1197(oracle, B, monkeypatch):
    w = wl.config2_units_pruned(B)
    weights, x = wl.make(w)
    pruned, _ = wl.prune_units(w, weights, 1197)
    ref = oracle.forward(pruned, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got, info = _run(w, pruned, x, None, None, expect_hc=1197)
    assert_close(got, ref, "bf16", w.name + " compacted")
    monkeypatch.setenv("LSTM_B200_COMPACT", "0")
    got, info = _run(w, pruned, x, None, None, expect_hc=0)
    assert_close(got, ref, "bf16", w.name + " zeros kept")


def test_default_policy_compacts_batches_only(oracle, monkeypatch):
    monkeypatch.delenv("LSTM_B200_COMPACT", raising=False)
    for B, hc in ((2, 0), (6, 50)):
        w = wl.Workload("rc_policy", 1, False, 20, 80, 3, B, "bf16", 0.3, seed=34)
        weights, x = wl.make(w)
        pruned, _ = wl.prune_units(w, weights, 50)
        ref = oracle.forward(pruned, x, layers=1, bidir=False, hidden=80)
        got, info = _run(w, pruned, x, None, None, expect_hc=hc)
        assert_close(got, ref, "bf16", f"policy B={B}")


def test_chunked_calls_on_a_compacted_handle_carry_state(oracle):
    w = wl.Workload("rc_chunk", 2, False, 20, 80, 9, 3, "bf16", 0.3, seed=33)
    weights, x = wl.make(w)
    pruned, _ = wl.prune_units(w, weights, 50)
    ref = oracle.forward(pruned, x, layers=2, bidir=False, hidden=80)
    assert_close(run_gpu(w, pruned, x, chunks=[4, 5]), ref, "bf16", "compacted chunked")
