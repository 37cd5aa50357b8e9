"""Layer-wavefront kernel against the oracle (needs a B200): unidirectional stacks of two to four layers run all
their layers in one launch, layer l on timestep t beside layer l-1 on t+1 (paper, Section 5.1: the language
model is two stacked recurrent layers).  The oracle needs nothing new: a stack is the composition of its
layers, which is one of its pins."""
import numpy as np
import pytest

import lstm_workloads as wl
from gpu_util import assert_close, run_gpu

pytestmark = pytest.mark.gpu


def small(name, L, in_dim, H, T, B, seed=1, scale=0.3):
    return wl.Workload(name, L, False, in_dim, H, T, B, "bf16", scale, seed=seed)


WAVE_SHAPES = [
    small("wave_h100_b1", 2, 40, 100, 6, 1),
    small("wave_h1_b1", 2, 3, 1, 4, 1),                         # one unit: most CTAs of each group own nothing
    small("wave_h149_b2_l3", 3, 64, 149, 5, 2),                 # three layers, two sequences
    small("wave_h64_b4_l4", 4, 20, 64, 7, 4),                   # four layers (37 CTAs each), four sequences
    small("wave_h300_t1", 2, 30, 300, 1, 3),                    # a single step: only initial states and the layer below
    small("wave_h700_b1", 2, 64, 700, 12, 1, scale=0.05),       # ten units per CTA, every tile in registers
    small("wave_h1000_b1", 2, 64, 1000, 8, 1, scale=0.04),      # the upper layer's slice spills into shared memory
    small("wave_h1024_b3", 2, 48, 1024, 4, 3, scale=0.03),      # the widest two-layer stack whose slices fit on-chip
    small("wave_h520_b2_l3", 3, 48, 520, 5, 2, scale=0.05),     # 49 CTAs per layer, eleven units each
]


@pytest.mark.parametrize("w", WAVE_SHAPES, ids=lambda w: w.name)
def test_wavefront_against_oracle(oracle, w, monkeypatch):
    import torch
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_WAVE", "1")
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=False, hidden=w.hidden)
    m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, dtype="bf16", max_T=w.T, max_B=w.B)
    assert m.info()["layer_wavefront"] == 1
    t = lambda a: torch.from_numpy(a).cuda()
    y, hT, cT = m.forward(t(x), t(h0), t(c0))
    m.check()
    assert m.info()["launches_per_forward"] == 3              # staging, layer 0's projection, the wavefront kernel
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", w.name)
    # a second call on the same handle (the slots of the first call carry older stamps), without initial states
    ref2 = oracle.forward(weights, x, layers=w.layers, bidir=False, hidden=w.hidden)
    y, hT, cT = m.forward(t(x))
    m.check()
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref2, "bf16", w.name + " second call")
    m.close()


def test_stacks_the_wavefront_kernel_does_not_serve_run_layer_by_layer(oracle, monkeypatch):
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_WAVE", "1")
    for w in (small("nowave_h1500", 2, 32, 1500, 2, 1, scale=0.03),          # 21 units per CTA of a half-GPU group
              small("nowave_h1184", 2, 32, 1184, 2, 1, scale=0.03),          # 16 units per CTA, but the slice exceeds shared memory
              wl.Workload("nowave_bidir", 2, True, 16, 64, 3, 1, "bf16", 0.3, seed=3),
              small("nowave_l1", 1, 16, 64, 3, 1)):
        weights, x = wl.make(w)
        ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
        m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype="bf16", max_T=w.T, max_B=w.B)
        assert m.info()["layer_wavefront"] == 0
        m.close()
        assert_close(run_gpu(w, weights, x), ref, "bf16", w.name)


def test_wavefront_and_layer_by_layer_agree_and_batches_fall_back(oracle, monkeypatch):
    """The same handle serves up to four sequences with the wavefront kernel and larger batches layer by layer."""
    import torch
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_WAVE", "1")
    w = small("wave_mixed", 2, 32, 200, 6, 9, seed=5)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=2, bidir=False, hidden=200)
    m = pkg.LSTM(weights, layers=2, in_dim=32, hidden=200, dtype="bf16", max_T=w.T, max_B=w.B)
    assert m.info()["layer_wavefront"] == 1
    xd = torch.from_numpy(x).cuda()
    y, hT, cT = m.forward(xd)
    m.check()
    assert m.info()["launches_per_forward"] == 5
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", "batch of nine")
    y, hT, cT = m.forward(xd[:, :3].contiguous())
    m.check()
    assert m.info()["launches_per_forward"] == 3
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), (ref[0][:, :3], ref[1][:, :3], ref[2][:, :3]), "bf16", "three of nine")
    m.close()


def test_wavefront_chunked_calls_carry_state(oracle, monkeypatch):
    monkeypatch.setenv("LSTM_B200_WAVE", "1")
    w = small("wave_chunk", 3, 24, 130, 11, 2, seed=6)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=3, bidir=False, hidden=130)
    assert_close(run_gpu(w, weights, x, chunks=[4, 1, 6]), ref, "bf16", "wave chunked")


def test_wavefront_withheld_words_end_in_a_timeout_status(oracle, monkeypatch):
    import torch
    import paper_1901_10997_b200 as pkg
    monkeypatch.setenv("LSTM_B200_WAVE", "1")
    w = small("wave_timeout", 2, 40, 300, 8, 2, seed=22)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=2, bidir=False, hidden=300)
    m = pkg.LSTM(weights, layers=2, in_dim=w.in_dim, hidden=w.hidden, dtype="bf16", max_T=w.T, max_B=w.B)
    assert m.info()["layer_wavefront"] == 1
    xd = torch.from_numpy(x).cuda()
    for cta in (5, 80):                          # a CTA of the lower layer's group, then one of the upper layer's
        m.selftest_timeout(cta, 2_000_000)
        m.forward(xd)
        assert m.status() == pkg.LSTM_ERR_TIMEOUT
        m.selftest_timeout(-1)
        y, hT, cT = m.forward(xd)
        m.check()
        assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", "after the timeout")
    m.close()
