"""H-LSTM cell on the GPU against the fp64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

import lstm_workloads as wl
from gpu_util import assert_close

pytestmark = pytest.mark.gpu


def run(w, Hh, weights, x, h0=None, c0=None):
    import torch
    import paper_1901_10997_b200 as pkg
    m = pkg.HLSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, gate_hidden=Hh, bidir=w.bidir,
                  dtype="bf16", max_T=w.T, max_B=w.B)
    try:
        dev = torch.device("cuda:0")
        h = torch.from_numpy(h0).to(dev) if h0 is not None else None
        c = torch.from_numpy(c0).to(dev) if c0 is not None else None
        y, hT, cT = m.forward(torch.from_numpy(x).to(dev), h, c)
        m.check()
        return y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()
    finally:
        m.close()


# (layers, bidir, in_dim, H, Hh, T, B, scale): H != Hh, sizes off every tile boundary, several batch rows
SHAPES = [
    (1, False, 5, 7, 9, 4, 1, 0.5),
    (2, True, 20, 33, 17, 5, 2, 0.4),
    (1, False, 64, 150, 200, 6, 3, 0.2),
    (2, False, 96, 300, 300, 5, 1, 0.15),
    (1, True, 40, 520, 260, 4, 2, 0.1),
    (1, False, 128, 1500, 1500, 3, 1, 0.03),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: f"L{s[0]}D{1 + s[1]}_in{s[2]}_H{s[3]}_Hh{s[4]}_T{s[5]}_B{s[6]}")
def test_hlstm_matches_oracle(oracle, shape):
    L, bidir, in_dim, H, Hh, T, B, scale = shape
    w = wl.Workload("hlstm", L, bidir, in_dim, H, T, B, "bf16", scale, seed=sum(shape[2:7]))
    weights, x = wl.make_hlstm(w, Hh)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward_hlstm(weights, x, h0, c0, layers=L, bidir=bidir, hidden=H, gate_hidden=Hh)
    assert_close(run(w, Hh, weights, x, h0, c0), ref, "bf16", "hlstm")


def test_hlstm_rejects_what_it_cannot_serve():
    import paper_1901_10997_b200 as pkg
    w = wl.Workload("hlstm", 1, False, 8, 16, 2, 1, "fp32", 0.1)
    weights, _ = wl.make_hlstm(w, 16)
    with pytest.raises(pkg.LstmError) as e:
        pkg.HLSTM(weights, layers=1, in_dim=8, hidden=16, gate_hidden=16, dtype="fp32", max_T=2, max_B=1)
    assert e.value.code == pkg.LSTM_ERR_UNSUPPORTED


def test_hlstm_withheld_words_end_in_a_timeout_status(oracle):
    """Both exchanges of the H-LSTM step (hidden-layer values, h) are bounded waits: a CTA that withholds
    its words makes the call end with LSTM_ERR_TIMEOUT, and the handle works again afterwards."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = wl.Workload("hlstm_timeout", 1, False, 24, 200, 6, 2, "bf16", 0.2, seed=77)
    weights, x = wl.make_hlstm(w, 160)
    ref = oracle.forward_hlstm(weights, x, layers=1, bidir=False, hidden=200, gate_hidden=160)
    m = pkg.HLSTM(weights, layers=1, in_dim=24, hidden=200, gate_hidden=160, dtype="bf16", max_T=w.T, max_B=w.B)
    xd = torch.from_numpy(x).cuda()
    m.selftest_timeout(3, 2_000_000)
    m.forward(xd)
    assert m.status() == pkg.LSTM_ERR_TIMEOUT
    m.selftest_timeout(-1)
    y, hT, cT = m.forward(xd)
    m.check()
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", "after the timeout")
    m.close()


def test_hlstm_chunked_calls_carry_state(oracle):
    import torch
    import paper_1901_10997_b200 as pkg
    w = wl.Workload("hlstm_chunks", 2, False, 30, 96, 10, 2, "bf16", 0.2, seed=78)
    weights, x = wl.make_hlstm(w, 80)
    ref = oracle.forward_hlstm(weights, x, layers=2, bidir=False, hidden=96, gate_hidden=80)
    m = pkg.HLSTM(weights, layers=2, in_dim=30, hidden=96, gate_hidden=80, dtype="bf16", max_T=8, max_B=2)
    xd = torch.from_numpy(x).cuda()
    y1, h, c = m.forward(xd[:4].contiguous())
    y2, h, c = m.forward(xd[4:].contiguous(), h, c)
    m.check()
    got = (torch.cat([y1, y2]).cpu().numpy(), h.cpu().numpy(), c.cpu().numpy())
    assert_close(got, ref, "bf16", "chunked")
    m.close()


def _fuzz_cases(n, seed):
    rng = np.random.default_rng(seed)
    return [dict(L=int(rng.integers(1, 3)), bidir=bool(rng.integers(0, 2)), in_dim=int(rng.integers(1, 150)),
                 H=int(rng.choice([rng.integers(1, 50), rng.integers(50, 600)])),
                 Hh=int(rng.choice([rng.integers(1, 50), rng.integers(50, 600)])),
                 T=int(rng.integers(1, 8)), B=int(rng.integers(1, 5)), seed=500 + i) for i in range(n)]


@pytest.mark.parametrize("c", _fuzz_cases(16, 77), ids=lambda c: "L{L}D{d}_in{in_dim}_H{H}_Hh{Hh}_T{T}_B{B}".format(d=1 + c["bidir"], **c))
def test_hlstm_random_shapes(oracle, c):
    scale = min(0.3, 2.0 / np.sqrt(max(c["H"], c["Hh"]) + c["in_dim"]))
    w = wl.Workload("hfuzz", c["L"], c["bidir"], c["in_dim"], c["H"], c["T"], c["B"], "bf16", scale, seed=c["seed"])
    weights, x = wl.make_hlstm(w, c["Hh"])
    h0, c0 = wl.make_states(w)
    ref = oracle.forward_hlstm(weights, x, h0, c0, layers=c["L"], bidir=c["bidir"], hidden=c["H"], gate_hidden=c["Hh"])
    assert_close(run(w, c["Hh"], weights, x, h0, c0), ref, "bf16", "hlstm fuzz")


def test_hlstm_keep_masks_equal_explicit_zeros(oracle):
    """Pruned H-LSTM (the model the paper ships, Table 1 row (d)): keep-masks given to the library against the
    oracle run on W (x) Msk written out; 80 % of every matrix pruned, two layers, both directions."""
    L, bidir, in_dim, H, Hh, T, B = 2, True, 24, 150, 130, 5, 2
    w = wl.Workload("hlstm_masked", L, bidir, in_dim, H, T, B, "bf16", 0.5, seed=77)
    weights, x = wl.make_hlstm(w, Hh)
    h0, c0 = wl.make_states(w)
    rng = np.random.default_rng(123)
    masked, zeroed = [], []
    for ws in weights:
        m = {k: (rng.random(ws[k].shape) < 0.2).astype(np.uint8) for k in ("ux", "uh", "w")}
        masked.append(dict(ws, mask_ux=m["ux"], mask_uh=m["uh"], mask_w=m["w"]))
        zeroed.append(dict(ws, ux=ws["ux"] * m["ux"], uh=ws["uh"] * m["uh"], w=ws["w"] * m["w"]))
    ref = oracle.forward_hlstm(zeroed, x, h0, c0, layers=L, bidir=bidir, hidden=H, gate_hidden=Hh)
    got = run(w, Hh, masked, x, h0, c0)
    assert_close(got, ref, "bf16", "hlstm/masks")
    dense_ref = oracle.forward_hlstm(weights, x, h0, c0, layers=L, bidir=bidir, hidden=H, gate_hidden=Hh)
    assert np.abs(dense_ref[0] - ref[0]).max() > 1e-2          # the masks change the result: they were applied
