"""lstm_forward_noalloc against lstm_forward and against the fp64 oracle (needs a B200).

The entry point under test serves callers that are not allowed to allocate device memory when they
run the model (fixed memory pools, an allocator owned by someone else): it works straight from the
caller's buffers and a scratch array that is part of the library image.  Because that array is shared
by every call and keeps what the previous call left in it, the check runs two calls in a row -- with
different inputs and shapes -- and compares each with the handle-based path through the C ABI.
This file sorts last so that a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest

import lstm_workloads as wl

pytestmark = pytest.mark.gpu


def _existing_path(pkg, torch, w, weights, x, h0, c0):
    m = pkg.LSTM(weights, layers=1, in_dim=w.in_dim, hidden=w.hidden, dtype="fp32", max_T=w.T, max_B=w.B)
    try:
        y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
        m.check()
        return y.cpu().numpy(), hT.cpu().numpy()[0], cT.cpu().numpy()[0]
    finally:
        m.close()


def _noalloc_path(pkg, torch, w, weights, x, h0, c0):
    dev = torch.device("cuda:0")
    t = {k: torch.from_numpy(np.ascontiguousarray(weights[0][k])).to(dev) for k in ("wx", "wh", "b")}
    xd, hd, cd = (torch.from_numpy(a).to(dev) for a in (x, h0[0], c0[0]))
    y = torch.full((w.T, w.B, w.hidden), float("nan"), device=dev)
    hT = torch.full((w.B, w.hidden), float("nan"), device=dev)
    cT = torch.full((w.B, w.hidden), float("nan"), device=dev)
    torch.cuda.synchronize()
    rc, msg = pkg.lstm_forward_noalloc(t["wx"].data_ptr(), t["wh"].data_ptr(), t["b"].data_ptr(), w.in_dim, w.hidden,
                                       xd.data_ptr(), w.T, w.B, hd.data_ptr(), cd.data_ptr(),
                                       y.data_ptr(), hT.data_ptr(), cT.data_ptr(),
                                       torch.cuda.current_stream().cuda_stream)
    assert rc == pkg.LSTM_OK, msg
    return y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()


def test_two_calls_in_a_row_match_the_handle_path(oracle):
    import torch
    import paper_1901_10997_b200 as pkg
    tol = wl.TOLERANCE["fp32"]
    # the second call is smaller in every dimension, so it runs over words the first one left behind
    for w in (wl.Workload("noalloc_a", 1, False, 45, 203, 9, 3, "fp32", 0.3, seed=31),
              wl.Workload("noalloc_b", 1, False, 20, 70, 5, 2, "fp32", 0.3, seed=32)):
        weights, x = wl.make(w)
        h0, c0 = wl.make_states(w)
        want = _existing_path(pkg, torch, w, weights, x, h0, c0)
        got = _noalloc_path(pkg, torch, w, weights, x, h0, c0)
        for name, g, r in zip(("y", "hT", "cT"), got, want):
            floored, scaled = wl.rel_err(g, r)
            assert floored <= tol, f"{w.name} {name}: {floored:.3e} (scaled {scaled:.3e}) > {tol}"
        # and against the independent CPU oracle, so that the two CUDA paths cannot be wrong together
        ref = oracle.forward(weights, x, h0, c0, layers=1, bidir=False, hidden=w.hidden)
        for name, g, r in zip(("y", "hT", "cT"), got, (ref[0], ref[1][0], ref[2][0])):
            floored, scaled = wl.rel_err(g, r)
            assert floored <= tol, f"{w.name} {name} vs oracle: {floored:.3e} (scaled {scaled:.3e}) > {tol}"


def test_sizes_beyond_the_built_in_scratch_are_rejected():
    import torch
    import paper_1901_10997_b200 as pkg
    d = torch.zeros(16, device="cuda")
    p = d.data_ptr()
    rc, msg = pkg.lstm_forward_noalloc(p, p, p, 8, 4097, p, 2, 2, 0, 0, p, 0, 0)     # B*H = 8194 > 8192
    assert rc == pkg.LSTM_ERR_UNSUPPORTED and "scratch" in msg
    rc, msg = pkg.lstm_forward_noalloc(p, p, p, 0, 4, p, 2, 2, 0, 0, p, 0, 0)
    assert rc == pkg.LSTM_ERR_INVALID


def test_withheld_words_end_in_a_timeout_not_a_hang(oracle, monkeypatch):
    """One CTA withholds its exchange words: the bounded waits of the others run out after a millisecond, the call
    returns LSTM_ERR_TIMEOUT, and the next call (the scratch array is cleared on entry) computes correctly."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = wl.Workload("noalloc_timeout", 1, False, 20, 70, 5, 2, "fp32", 0.3, seed=33)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    dev = torch.device("cuda:0")
    t = {k: torch.from_numpy(np.ascontiguousarray(weights[0][k])).to(dev) for k in ("wx", "wh", "b")}
    xd, hd, cd = (torch.from_numpy(a).to(dev) for a in (x, h0[0], c0[0]))
    y = torch.zeros((w.T, w.B, w.hidden), device=dev)
    args = (t["wx"].data_ptr(), t["wh"].data_ptr(), t["b"].data_ptr(), w.in_dim, w.hidden, xd.data_ptr(), w.T, w.B,
            hd.data_ptr(), cd.data_ptr(), y.data_ptr(), 0, 0, torch.cuda.current_stream().cuda_stream)
    monkeypatch.setenv("LSTM_B200_NOALLOC_SELFTEST", "3:2000000")
    rc, msg = pkg.lstm_forward_noalloc(*args)
    assert rc == pkg.LSTM_ERR_TIMEOUT and "timeout" in msg
    monkeypatch.delenv("LSTM_B200_NOALLOC_SELFTEST")
    ref = oracle.forward(weights, x, h0, c0, layers=1, bidir=False, hidden=w.hidden)
    got = _noalloc_path(pkg, torch, w, weights, x, h0, c0)
    floored, scaled = wl.rel_err(got[0], ref[0])
    assert floored <= wl.TOLERANCE["fp32"], (floored, scaled)
