"""Pin of the identity behind the compacted format for row/column-pruned stacks (paper, Section 4.2,
Algorithm 1: whole rows and columns of the gate matrices are zero, which shrinks the model's dimension).

A hidden unit whose four gate rows are zero and whose outgoing columns are zero reads nothing and is read by
nobody.  Then (a) the remaining units form a smaller LSTM whose results are those of the full model with the
zeros left in, and (b) the removed unit's own state follows from its bias alone: constant gates,
c_t = f c_{t-1} + i g, h_t = o tanh(c_t).  Both are checked on the oracle, in fp64, with the compaction and the
closed form written out here independently of the library (CPU only)."""
import numpy as np
import pytest

import lstm_workloads as wl


def _compact_model(w, weights, removed):
    """The smaller model over the surviving units of every (layer, direction), by plain indexing."""
    H, D = w.hidden, w.dirs
    keep = [np.setdiff1d(np.arange(H), r) for r in removed]
    out = []
    for l in range(w.layers):
        for d in range(D):
            e = weights[l * D + d]
            k = keep[l * D + d]
            rows = (np.arange(4)[:, None] * H + k[None, :]).ravel()
            if l == 0:
                cols = np.arange(w.in_dim)
            else:
                cols = np.concatenate([d2 * H + keep[(l - 1) * D + d2] for d2 in range(D)])
            out.append({"wx": e["wx"][np.ix_(rows, cols)].copy(), "wh": e["wh"][np.ix_(rows, k)].copy(), "b": e["b"][rows].copy()})
    return out, keep


def _sigma(z):
    return 1.0 / (1.0 + np.exp(-z))


@pytest.mark.parametrize("layers,bidir", [(1, False), (2, False), (2, True), (3, True)])
def test_surviving_units_form_a_smaller_model_and_removed_units_follow_their_bias(oracle, layers, bidir):
    H, keep_n, T, B = 12, 7, 6, 3
    w = wl.Workload("rc", layers, bidir, 5, H, T, B, "fp32", 0.6, seed=77 + layers)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    pruned, removed = wl.prune_units(w, weights, keep_n)
    D = w.dirs
    y, hT, cT = oracle.forward(pruned, x, h0, c0, layers=layers, bidir=bidir, hidden=H)

    small, keep = _compact_model(w, pruned, removed)
    # every (layer, direction) removes the same NUMBER of units here, so the compact model has one width
    h0s = np.stack([h0[i][:, keep[i]] for i in range(layers * D)])
    c0s = np.stack([c0[i][:, keep[i]] for i in range(layers * D)])
    ys, hTs, cTs = oracle.forward(small, x, h0s, c0s, layers=layers, bidir=bidir, hidden=keep_n)
    for d in range(D):
        k = keep[(layers - 1) * D + d]
        assert np.array_equal(y[:, :, d * H + k], ys[:, :, d * keep_n:(d + 1) * keep_n])       # adding 0 * h changes no sum
    for i in range(layers * D):
        assert np.array_equal(hT[i][:, keep[i]], hTs[i]) and np.array_equal(cT[i][:, keep[i]], cTs[i])

    # removed units: constant gates from the bias, state from c0 alone
    for i in range(layers * D):
        l, d = divmod(i, D)
        b = pruned[i]["b"].astype(np.float64)
        for j in removed[i]:
            gi, gf, gg, go = _sigma(b[j]), _sigma(b[H + j]), np.tanh(b[2 * H + j]), _sigma(b[3 * H + j])
            c = c0[i][:, j].astype(np.float64)
            for s in range(T):
                c = gf * c + gi * gg
                h = go * np.tanh(c)
                if l == layers - 1:
                    t = T - 1 - s if d == 1 else s
                    np.testing.assert_allclose(y[t, :, d * H + j], h, rtol=1e-12, atol=1e-15)
            np.testing.assert_allclose(hT[i][:, j], h, rtol=1e-12, atol=1e-15)
            np.testing.assert_allclose(cT[i][:, j], c, rtol=1e-12, atol=1e-15)


def test_a_unit_that_is_still_read_may_not_be_removed(oracle):
    """The identity needs BOTH halves: zero rows alone (the unit still feeds others through its column of Wh)
    leave a unit whose constant-gate output the other units depend on; dropping it changes their results."""
    H, T, B = 6, 5, 2
    w = wl.Workload("rc_read", 1, False, 4, H, T, B, "fp32", 0.8, seed=5)
    weights, x = wl.make(w)
    j = 2
    e = weights[0]
    rows = np.arange(4) * H + j
    e["wx"][rows] = 0.0
    e["wh"][rows] = 0.0                     # rows zero, column of wh NOT zero
    y, _, _ = oracle.forward(weights, x, layers=1, bidir=False, hidden=H)
    keep = np.setdiff1d(np.arange(H), [j])
    r = (np.arange(4)[:, None] * H + keep[None, :]).ravel()
    small = [{"wx": e["wx"][r], "wh": e["wh"][np.ix_(r, keep)], "b": e["b"][r]}]
    ys, _, _ = oracle.forward(small, x, layers=1, bidir=False, hidden=H - 1)
    assert np.max(np.abs(y[:, :, keep] - ys)) > 1e-3
