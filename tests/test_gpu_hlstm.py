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
