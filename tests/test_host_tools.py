"""Host-side helpers of the library (no GPU): latency-hysteresis analysis of a measured curve (paper,
Section 3) and folding of an inter-layer affine map into the next layer's input weights (Section 5.2).
Each is checked against the definition written out here by brute force."""
import numpy as np
import pytest

import paper_1901_10997_b200 as pkg


def dominated(sizes, lat, i, eps):
    """Section 3: a size is inside a hysteresis bin when some LARGER size is at least as fast."""
    return any(sizes[j] > sizes[i] and lat[j] <= lat[i] * (1 + eps) for j in range(len(sizes)))


CURVE_SIZES = [128, 136, 144, 152, 160, 168, 176, 184, 192, 200]
CURVE_LAT = [50.0, 50.0, 49.0, 61.0, 60.0, 60.5, 60.0, 72.0, 71.0, 71.0]     # three plateaus (staircase)


def test_staircase_has_one_lhp_per_plateau():
    rc, flags, count = pkg.lstm_lhp_points(CURVE_SIZES, CURVE_LAT, 0.0)
    assert rc == pkg.LSTM_OK
    lhps = [s for s, f in zip(CURVE_SIZES, flags) if f]
    # the right end of each plateau: 144 (49 < everything after), 176 (60 < 71), 200 (largest size)
    assert lhps == [144, 176, 200] and count == 3
    # redundancy of the architecture space, (1 - #LHP / #points) * 100 %
    assert (1 - count / len(CURVE_SIZES)) * 100 == pytest.approx(70.0)


def test_eps_merges_nearly_equal_latencies():
    sizes, lat = [100, 200, 300], [10.0, 10.04, 20.0]
    assert pkg.lstm_lhp_points(sizes, lat, 0.0)[1] == [1, 1, 1]          # 10.0 < 10.04: strictly faster
    assert pkg.lstm_lhp_points(sizes, lat, 0.005)[1] == [0, 1, 1]        # within 0.5 %: the larger one wins


@pytest.mark.parametrize("seed", range(8))
def test_lhp_points_match_the_definition_on_random_curves(seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(1, 40))
    sizes = rng.permutation(np.arange(8, 8 + 8 * 60, 8))[:n].tolist()     # unsorted on purpose
    lat = (np.floor(np.array(sizes) / 64.0) * 5 + 20 + rng.normal(0, 0.4, n)).tolist()
    for eps in (0.0, 0.005, 0.05):
        rc, flags, count = pkg.lstm_lhp_points(sizes, lat, eps)
        assert rc == pkg.LSTM_OK
        want = [0 if dominated(sizes, lat, i, eps) else 1 for i in range(n)]
        assert flags == want and count == sum(want)
        assert flags[int(np.argmax(sizes))] == 1                           # the largest size is never dominated


def test_nearest_lhp_is_the_growth_target():
    # a model pruned to 150 is grown back to the next size that no larger model beats
    assert pkg.lstm_nearest_lhp(CURVE_SIZES, CURVE_LAT, 150) == (pkg.LSTM_OK, 176)
    assert pkg.lstm_nearest_lhp(CURVE_SIZES, CURVE_LAT, 144) == (pkg.LSTM_OK, 144)
    assert pkg.lstm_nearest_lhp(CURVE_SIZES, CURVE_LAT, 1) == (pkg.LSTM_OK, 144)
    assert pkg.lstm_nearest_lhp(CURVE_SIZES, CURVE_LAT, 177) == (pkg.LSTM_OK, 200)
    rc, _ = pkg.lstm_nearest_lhp(CURVE_SIZES, CURVE_LAT, 201)
    assert rc == pkg.LSTM_ERR_UNSUPPORTED


@pytest.mark.parametrize("seed", range(4))
def test_nearest_lhp_matches_brute_force(seed):
    rng = np.random.default_rng(2000 + seed)
    sizes = list(range(16, 400, 8))
    lat = (np.ceil(np.array(sizes) / 48.0) * 3 + rng.normal(0, 0.2, len(sizes))).tolist()
    for req in (16, 50, 123, 300, 392):
        cands = [s for i, s in enumerate(sizes) if s >= req and not dominated(sizes, lat, i, 0.01)]
        assert pkg.lstm_nearest_lhp(sizes, lat, req, 0.01) == (pkg.LSTM_OK, min(cands))


def test_lhp_rejects_malformed_curves():
    assert pkg.lstm_lhp_points([], [], 0.0)[0] == pkg.LSTM_ERR_INVALID
    assert pkg.lstm_lhp_points([8, 8], [1.0, 2.0], 0.0)[0] == pkg.LSTM_ERR_INVALID        # repeated size
    assert pkg.lstm_lhp_points([8, 16], [1.0, 0.0], 0.0)[0] == pkg.LSTM_ERR_INVALID       # non-positive latency
    assert pkg.lstm_lhp_points([8, 16], [1.0, float("nan")], 0.0)[0] == pkg.LSTM_ERR_INVALID
    assert pkg.lstm_lhp_points([8, 16], [1.0, 2.0], -0.1)[0] == pkg.LSTM_ERR_INVALID
    assert pkg.lstm_lhp_points([0, 16], [1.0, 2.0], 0.0)[0] == pkg.LSTM_ERR_INVALID


def test_fold_input_affine_is_the_identity_it_claims():
    """Wx (s * x + t) + b == (Wx diag(s)) x + (b + Wx t) for every x (checked in float64)."""
    rng = np.random.default_rng(7)
    rows, cols = 24, 11
    wx = rng.uniform(-1, 1, (rows, cols)).astype(np.float32)
    b = rng.uniform(-1, 1, rows).astype(np.float32)
    s = rng.uniform(0.5, 2.0, cols).astype(np.float32)
    t = rng.uniform(-1, 1, cols).astype(np.float32)
    rc, wf, bf = pkg.lstm_fold_input_affine(wx, b, s, t)
    assert rc == pkg.LSTM_OK and wf.dtype == np.float32 and wf.shape == wx.shape and bf.shape == (rows,)
    for _ in range(5):
        x = rng.normal(0, 1, cols)
        want = wx.astype(np.float64) @ (s.astype(np.float64) * x + t.astype(np.float64)) + b
        got = wf.astype(np.float64) @ x + bf
        np.testing.assert_allclose(got, want, rtol=0, atol=5e-6)
    # element-wise: a column scale, nothing transposed
    np.testing.assert_array_equal(wf, wx * s[None, :])


def test_fold_defaults_and_errors():
    wx = np.arange(6, dtype=np.float32).reshape(2, 3)
    rc, wf, bf = pkg.lstm_fold_input_affine(wx, None, None, None)
    assert rc == pkg.LSTM_OK
    np.testing.assert_array_equal(wf, wx)
    np.testing.assert_array_equal(bf, np.zeros(2, np.float32))
    rc, wf, bf = pkg.lstm_fold_input_affine(wx, None, None, np.array([1, 1, 1], np.float32))
    np.testing.assert_array_equal(bf, wx.sum(axis=1))                      # shift only: bias picks up the row sums
    lib = pkg.load_library()
    assert lib.lstm_fold_input_affine(None, None, 2, 3, None, None, None, None) == pkg.LSTM_ERR_INVALID
