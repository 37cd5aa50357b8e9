"""A frozen batch-normalisation (per-feature scale and shift) between two recurrent layers (paper,
Section 5.2), folded into the second layer's input weights with lstm_fold_input_affine, gives the same
outputs as the oracle run layer by layer with the affine map applied explicitly in float64."""
import numpy as np
import pytest

import lstm_workloads as wl
import paper_1901_10997_b200 as pkg
from gpu_util import assert_close, run_gpu

pytestmark = pytest.mark.gpu


def oracle_with_affine(oracle, w, weights, x, scale, shift):
    D, H = (2 if w.bidir else 1), w.hidden
    y0, h0T, c0T = oracle.forward(weights[:D], x, layers=1, bidir=w.bidir, hidden=H)
    x1 = y0 * scale.astype(np.float64)[None, None, :] + shift.astype(np.float64)[None, None, :]
    y1, h1T, c1T = oracle.forward(weights[D:], x1, layers=1, bidir=w.bidir, hidden=H)
    return y1, np.concatenate([h0T, h1T]), np.concatenate([c0T, c1T])


@pytest.mark.parametrize("dtype,bidir,H,B", [("fp32", True, 37, 3), ("bf16", False, 200, 2), ("bf16", True, 150, 6)])
def test_folded_affine_matches_explicit_one(oracle, dtype, bidir, H, B):
    w = wl.Workload("fold", 2, bidir, 19, H, 6, B, dtype, 0.1, seed=77)
    weights, x = wl.make(w)
    D = 2 if bidir else 1
    rng = np.random.default_rng(5)
    if dtype == "bf16":
        # powers of two keep the folded weights exactly representable in bf16, so that the rounding of the
        # folded matrix (which the oracle, applying the map to the activations, never sees) is not counted
        scale = np.exp2(rng.integers(-1, 2, D * H)).astype(np.float32)
    else:
        scale = rng.uniform(0.5, 1.5, D * H).astype(np.float32)
    shift = rng.uniform(-0.3, 0.3, D * H).astype(np.float32)
    ref = oracle_with_affine(oracle, w, weights, x, scale, shift)
    folded = [dict(s) for s in weights]
    for d in range(D):
        rc, wx, b = pkg.lstm_fold_input_affine(weights[D + d]["wx"], weights[D + d].get("b"), scale, shift)
        assert rc == pkg.LSTM_OK
        folded[D + d]["wx"], folded[D + d]["b"] = wx, b
    got = run_gpu(w, folded, x)
    assert_close(got, ref, dtype, f"fold/{dtype}")
    # and the fold matters: without it the second layer sees different inputs
    plain = run_gpu(w, weights, x)
    floored, _ = wl.rel_err(plain[0], ref[0])
    assert floored > 10 * wl.TOLERANCE[dtype]
