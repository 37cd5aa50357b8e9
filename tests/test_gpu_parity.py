"""CUDA library vs fp64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

import lstm_workloads as wl
from gpu_util import assert_close, csr_weights, run_gpu

pytestmark = pytest.mark.gpu


def small(name, L, bidir, in_dim, H, T, B, dtype, density=1.0, seed=1, scale=0.3):
    return wl.Workload(name, L, bidir, in_dim, H, T, B, dtype, scale, density=density, seed=seed)


# awkward shapes: H not a multiple of 8/32/148, H = 1, T = 1, B not a power of two, in != H
SHAPES = [
    small("h1", 1, False, 1, 1, 3, 1, "fp32"),
    small("h2_bidir", 2, True, 3, 2, 3, 2, "fp32"),
    small("h7_b3", 2, False, 5, 7, 4, 3, "fp32"),
    small("t1", 1, True, 9, 33, 1, 5, "bf16"),
    small("h100_b1", 1, False, 40, 100, 6, 1, "bf16"),
    small("h149_b2", 2, False, 64, 149, 5, 2, "bf16"),
    small("h300_b5", 1, True, 77, 300, 7, 5, "bf16"),
    small("h300_b16", 1, False, 96, 300, 5, 16, "fp32"),
    small("h200_b20", 3, True, 50, 200, 4, 20, "bf16"),
    small("h513_b9", 1, False, 130, 513, 3, 9, "bf16"),
    # register-resident kernel with part of the slice in shared memory, several batch rows (register polling)
    small("h1896_b3", 1, False, 72, 1896, 3, 3, "bf16", scale=0.03),      # weights ~ 1/sqrt(H) as in the sweep
    # two passes of four rows with the staged exchange, both directions
    small("h640_b7", 1, True, 48, 640, 4, 7, "bf16"),
]


@pytest.mark.parametrize("w", SHAPES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", ["dense", "csr"])
def test_small_shapes(oracle, w, mode):
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got = run_gpu(w, weights, x, h0, c0, exec_mode=mode)
    assert_close(got, ref, w.dtype, f"{w.name}/{mode}")


@pytest.mark.parametrize("mode", ["dense", "csr"])
def test_masked_small(oracle, mode):
    w = small("masked", 2, True, 60, 90, 6, 3, "bf16", density=0.2, seed=5)
    weights, x = wl.make(w)
    weights[0]["mask_h"][5] = 0                      # an empty recurrent row
    weights[0]["wh"][5] = 0
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got = run_gpu(w, weights if mode == "dense" else csr_weights(oracle, weights), x, exec_mode=mode)
    assert_close(got, ref, w.dtype, mode)


def test_masks_apply_as_zeros_in_dense_mode(oracle):
    """A mask handed to the dense path multiplies the weights (W (x) Msk), it is not ignored."""
    w = small("maskapply", 1, False, 20, 24, 5, 2, "fp32", seed=6)
    weights, x = wl.make(w)
    rng = np.random.default_rng(1)
    mx = (rng.random(weights[0]["wx"].shape) < 0.5).astype(np.uint8)
    mh = (rng.random(weights[0]["wh"].shape) < 0.5).astype(np.uint8)
    masked = [{**weights[0], "mask_x": mx, "mask_h": mh}]
    ref = oracle.forward(masked, x, layers=1, bidir=False, hidden=w.hidden)
    for mode in ("dense", "csr"):
        assert_close(run_gpu(w, masked, x, exec_mode=mode), ref, "fp32", mode)


def test_chunked_calls_carry_state(oracle):
    w = small("chunk", 2, False, 30, 70, 12, 3, "bf16", seed=7)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=2, bidir=False, hidden=w.hidden)
    got = run_gpu(w, weights, x, chunks=[5, 1, 6])
    assert_close(got, ref, "bf16", "chunked")
    wb = w.with_(bidir=True, layers=1)
    weights, x = wl.make(wb)
    h0, c0 = wl.make_states(wb)
    ref = oracle.forward(weights, x, h0, c0, layers=1, bidir=True, hidden=w.hidden)
    assert_close(run_gpu(wb, weights, x, h0, c0, max_T=20, max_B=6), ref, "bf16", "larger workspace")


def test_empty_sequence_and_batch(oracle):
    import torch
    import paper_1901_10997_b200 as pkg
    w = small("empty", 1, False, 4, 6, 3, 2, "fp32")
    weights, x = wl.make(w)
    m = pkg.LSTM(weights, layers=1, in_dim=4, hidden=6, dtype="fp32", max_T=4, max_B=2)
    h0, c0 = wl.make_states(w)
    h = torch.from_numpy(h0).cuda(); c = torch.from_numpy(c0).cuda()
    y, hT, cT = m.forward(torch.empty((0, 2, 4), device="cuda"), h, c)
    m.check()
    assert y.shape == (0, 2, 6) and torch.equal(hT, h) and torch.equal(cT, c)
    y, hT, cT = m.forward(torch.empty((3, 0, 4), device="cuda"))
    m.check()
    assert y.shape == (3, 0, 6)
    with pytest.raises(pkg.LstmError):
        m.forward(torch.zeros((5, 2, 4), device="cuda"))          # T > max_T
    with pytest.raises(pkg.LstmError):
        m.forward(torch.zeros((1, 3, 4), device="cuda"))          # B > max_B
    m.close()


def test_bad_csr_is_rejected():
    import paper_1901_10997_b200 as pkg
    H, in_dim = 3, 2
    rp = np.array([0, 2] + [2] * (4 * H - 1), np.int32)
    bad = {"wx_csr": (rp, np.array([1, 0], np.int32), np.ones(2, np.float32)),     # unsorted columns
           "wh": np.zeros((4 * H, H), np.float32)}
    with pytest.raises(pkg.LstmError) as e:
        pkg.LSTM([bad], layers=1, in_dim=in_dim, hidden=H, dtype="fp32", exec_mode="csr", max_T=2, max_B=1)
    assert e.value.code == pkg.LSTM_ERR_INVALID
    bad["wx_csr"] = (rp, np.array([0, 7], np.int32), np.ones(2, np.float32))          # out of range
    with pytest.raises(pkg.LstmError):
        pkg.LSTM([bad], layers=1, in_dim=in_dim, hidden=H, dtype="fp32", exec_mode="csr", max_T=2, max_B=1)


def test_host_buffer_call_matches_device_call(oracle):
    import paper_1901_10997_b200 as pkg
    w = small("host", 2, False, 33, 65, 6, 4, "bf16", seed=9)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=2, bidir=False, hidden=w.hidden)
    m = pkg.LSTM(weights, layers=2, in_dim=w.in_dim, hidden=w.hidden, dtype="bf16", max_T=w.T, max_B=w.B)
    got = m.forward_host(x, h0, c0)
    assert_close(got, ref, "bf16", "host")
    m.close()


# ---------------------------------------------------------------- the five configurations
def test_config1_full(oracle):
    w = wl.config1()
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


def test_config2_b1_full(oracle):
    w = wl.config2(1)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


def test_config2_b20_every_column(oracle):
    """Full size on both sides: all 20 batch columns against the oracle (columns are independent in the
    mathematics, not in the kernel, which reads its accumulator in chunks of 16 columns)."""
    w = wl.config2(20)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


@pytest.mark.parametrize("H", wl.config3_sizes())
def test_config3_points(oracle, H):
    """Every size of the hidden-width sweep is a correct model, not only the ones on a tile boundary."""
    w = wl.config3(H)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=1, bidir=False, hidden=H)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


@pytest.mark.parametrize("density", [0.10, 0.05])
def test_config4_dense_with_zeros_vs_csr(oracle, density):
    w = wl.config4(density)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    dense = run_gpu(w, weights, x, exec_mode="dense")
    sparse = run_gpu(w, weights, x, exec_mode="csr")
    assert_close(dense, ref, w.dtype, "dense-with-zeros")
    assert_close(sparse, ref, w.dtype, "csr")
    assert_close(sparse, dense, w.dtype, "csr vs dense")


def test_config5_b1_full(oracle):
    w = wl.config5(1)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


def test_config5_b16_every_column(oracle):
    """All 16 utterances of the speech-shaped stack against the oracle (the slowest oracle run of the suite:
    about a teraflop of fp64 loops over the host cores)."""
    w = wl.config5(16)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    assert_close(run_gpu(w, weights, x), ref, w.dtype, w.name)


# ---------------------------------------------------------------- kernel selection and the failure path
def test_shared_memory_kernel_serves_bf16_dense_when_selected(oracle, monkeypatch):
    """bf16 dense weights normally run on the register-resident kernel; the shared-memory kernel is its
    fall-back for slices that do not fit and must stay correct."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = small("simt_bf16", 2, True, 64, 149, 6, 3, "bf16", seed=21)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    for env, resident in (("simt", 0), ("", 1)):
        monkeypatch.setenv("LSTM_B200_RECUR", env)
        m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=True, dtype="bf16",
                     max_T=w.T, max_B=w.B)
        assert m.info()["recur_register_resident"] == resident
        y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
        m.check()
        assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"recur={env or 'default'}")
        m.close()


# batches of 5..32 sequences on bf16 dense handles run the batched tensor-core recurrence: its edges
TC_SHAPES = [
    small("tc_h7_b6", 1, True, 5, 7, 3, 6, "bf16"),                 # one K block, a few rows per CTA, most CTAs with one unit
    small("tc_h64_b5_t1", 1, False, 20, 64, 1, 5, "bf16"),          # a single step: only the published h0 is consumed
    small("tc_h129_b32", 1, False, 33, 129, 4, 32, "bf16"),         # the largest batch (N = 64), ragged K tail of one column
    small("tc_h1000_b17", 2, False, 64, 1000, 3, 17, "bf16", scale=0.05),   # 16 K blocks, four per stage; two layers
    small("tc_h1600_b9", 1, False, 32, 1600, 2, 9, "bf16", scale=0.03),     # 25 K blocks: the ring is down to a few stages
    small("tc_h600_b32", 1, True, 24, 600, 3, 32, "bf16", scale=0.05),      # cluster pairs, both directions
    small("tc_h300_b64", 2, True, 24, 300, 3, 64, "bf16", scale=0.05),      # the largest batch (N = 128): two rounds of accumulator chunks
    small("tc_h1500_b48", 1, False, 40, 1500, 2, 48, "bf16", scale=0.03),   # N = 96 beside the full-width slice: two-block stages
    small("tc_h1500_b64", 1, False, 40, 1500, 2, 64, "bf16", scale=0.03),   # N = 128 beside the full-width slice: one-block stages
    small("tc_h592_b6_t1", 1, False, 16, 592, 1, 6, "bf16", scale=0.05),    # cluster pairs, a single step, uneven K halves (10 blocks: 5 + 5; 592 = 9.25 blocks)
    # 14 units per CTA x 32 K blocks do not fit shared memory: the handle keeps the register-resident kernel
    small("notc_h2000_b9", 1, False, 32, 2000, 2, 9, "bf16", scale=0.03),
]


@pytest.mark.parametrize("w", TC_SHAPES, ids=lambda w: w.name)
def test_batched_tensor_core_recurrence(oracle, w):
    import torch
    import paper_1901_10997_b200 as pkg
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype="bf16", max_T=w.T, max_B=w.B)
    assert bool(m.info()["recur_batched_tensor_core"]) == (not w.name.startswith("notc"))
    y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
    m.check()
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", w.name)
    # a smaller batch on the same handle goes through the register-resident kernel and must agree too
    if w.B > 6:
        nb = 3
        xs, hs, cs = x[:, :nb].copy(), h0[:, :nb].copy(), c0[:, :nb].copy()
        y2, h2, c2 = m.forward(torch.from_numpy(xs).cuda(), torch.from_numpy(hs).cuda(), torch.from_numpy(cs).cuda())
        m.check()
        assert_close((y2.cpu().numpy(), h2.cpu().numpy(), c2.cpu().numpy()), (ref[0][:, :nb], ref[1][:, :nb], ref[2][:, :nb]), "bf16", w.name + "/b3")
    m.close()


@pytest.mark.parametrize("B", [6, 20])
def test_first_call_of_a_fresh_handle_sees_a_nonzero_initial_state(oracle, B):
    """The batched kernel publishes h0 under the call's first stamp; on a fresh handle (cleared flags and
    planes) a consumer must still wait for that stamp instead of taking the cleared planes for h0.  Several
    fresh handles in a row, one step each, so that a CTA that starts early would read zeros."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = small("fresh_h0", 1, False, 24, 600, 1, B, "bf16", scale=0.05, seed=41)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=1, bidir=False, hidden=w.hidden)
    for _ in range(4):
        m = pkg.LSTM(weights, layers=1, in_dim=w.in_dim, hidden=w.hidden, dtype="bf16", max_T=w.T, max_B=w.B)
        assert m.info()["recur_batched_tensor_core"] >= 1
        y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
        m.check()
        assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"fresh handle B={B}")
        m.close()


@pytest.mark.parametrize("B", [2, 9])
def test_wide_bidirectional_stack_runs_its_directions_one_after_the_other(oracle, B):
    """At this width half the SMs cannot hold one direction's slice on-chip, so the handle gives each
    direction all SMs in turn (148 CTAs per direction instead of 74); results are the same stack."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = small("seq_dirs", 2, True, 40, 1500, 3, B, "bf16", scale=0.03, seed=31)
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w)
    ref = oracle.forward(weights, x, h0, c0, layers=2, bidir=True, hidden=w.hidden)
    m = pkg.LSTM(weights, layers=2, in_dim=w.in_dim, hidden=w.hidden, bidir=True, dtype="bf16", max_T=w.T, max_B=B)
    info = m.info()
    assert info["ctas_per_dir"] == info["sm_count"] and info["recur_register_resident"] == 1
    y, hT, cT = m.forward(torch.from_numpy(x).cuda(), torch.from_numpy(h0).cuda(), torch.from_numpy(c0).cuda())
    m.check()
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"seq dirs B={B}")
    m.close()


def test_batched_recurrence_chunked_calls_carry_state(oracle):
    w = small("tc_chunk", 2, True, 24, 150, 9, 8, "bf16", seed=9)
    weights, x = wl.make(w)
    # state carried across calls is only defined for one direction per call order; use the forward stack
    wf = w.with_(bidir=False)
    weights, x = wl.make(wf)
    ref = oracle.forward(weights, x, layers=2, bidir=False, hidden=wf.hidden)
    assert_close(run_gpu(wf, weights, x, chunks=[4, 1, 4]), ref, "bf16", "tc chunked")


@pytest.mark.parametrize("dtype,mode,B", [("bf16", "dense", 2), ("fp32", "dense", 2), ("bf16", "csr", 2), ("bf16", "dense", 6)])
def test_withheld_exchange_words_end_in_a_timeout_status_not_a_hang(oracle, dtype, mode, B):
    """One CTA withholds its h values (B = 6: its stamp, in the batched kernel); the waits of the others run
    out after a millisecond, the call reports LSTM_ERR_TIMEOUT, and the same handle computes correctly
    again afterwards."""
    import torch
    import paper_1901_10997_b200 as pkg
    w = small("timeout", 1, False, 40, 300, 8, B, dtype, seed=22)
    weights, x = wl.make(w)
    ref = oracle.forward(weights, x, layers=1, bidir=False, hidden=w.hidden)
    m = pkg.LSTM(weights, layers=1, in_dim=w.in_dim, hidden=w.hidden, dtype=dtype, exec_mode=mode, max_T=w.T, max_B=w.B)
    xd = torch.from_numpy(x).cuda()
    m.selftest_timeout(5, 2_000_000)              # about a millisecond of clock ticks
    m.forward(xd)
    assert m.status() == pkg.LSTM_ERR_TIMEOUT
    assert "timeout" in pkg.lstm_last_error(m.handle)
    m.selftest_timeout(-1)
    y, hT, cT = m.forward(xd)
    m.check()
    assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, dtype, "after the timeout")
    m.close()


# ---------------------------------------------------------------- the input projection on its own
@pytest.mark.parametrize("case", [("bf16", "dense", 1.0), ("bf16", "dense", 0.1), ("bf16", "csr", 0.1), ("fp32", "dense", 1.0),
                                  ("fp32", "csr", 0.3)], ids=lambda c: f"{c[0]}-{c[1]}-{c[2]}")
@pytest.mark.parametrize("shape", [(1, 7, 9, 3, 2), (2, 200, 136, 5, 3), (1, 1500, 375, 16, 1), (2, 1312, 200, 40, 4)],
                         ids=lambda s: f"D{s[0]}_in{s[1]}_H{s[2]}_T{s[3]}_B{s[4]}")
def test_input_projection_alone(oracle, case, shape):
    """Tensor-core, CUDA-core and CSR projections against the matrix product written out, ragged in every
    dimension (rows, columns, K tail), with split-K (short sequences) and without."""
    import torch
    import paper_1901_10997_b200 as pkg
    dtype, mode, density = case
    D, in_dim, H, T, B = shape
    w = wl.Workload("proj", 1, D == 2, in_dim, H, T, B, dtype, 0.2, density=density, seed=in_dim + H)
    weights, x = wl.make(w)
    ref = oracle.input_projection(weights, x, bidir=D == 2, hidden=H)
    m = pkg.LSTM(weights, layers=1, in_dim=in_dim, hidden=H, bidir=D == 2, dtype=dtype, exec_mode=mode, max_T=T, max_B=B)
    g = m.input_projection(torch.from_numpy(x).cuda())
    m.check()
    floored, scaled = wl.rel_err(g.cpu().numpy(), ref)
    # one rounding of each activation term (bf16 hi + lo, about 2^-17) or fp32 storage of the result
    assert scaled <= (1e-4 if dtype == "bf16" else 1e-6), (floored, scaled)
    m.close()


# ---------------------------------------------------------------- seeded random shapes
def _fuzz_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        H = int(rng.choice([rng.integers(1, 40), rng.integers(40, 300), rng.integers(300, 900)]))
        cases.append(dict(L=int(rng.integers(1, 3)), bidir=bool(rng.integers(0, 2)), in_dim=int(rng.integers(1, 200)), H=H,
                          T=int(rng.integers(1, 10)), B=int(rng.integers(1, 10)), dtype=str(rng.choice(["bf16", "bf16", "fp32"])),
                          mode=str(rng.choice(["dense", "dense", "csr"])), states=bool(rng.integers(0, 2)),
                          density=float(rng.choice([1.0, 0.3])), seed=1000 + i))
    return cases


@pytest.mark.parametrize("c", _fuzz_cases(36, 2024), ids=lambda c: "L{L}D{d}_in{in_dim}_H{H}_T{T}_B{B}_{dtype}_{mode}".format(d=1 + c["bidir"], **c))
def test_random_shapes(oracle, c):
    """Shapes nobody picked by hand: every kernel variant (register-resident, shared-memory, CSR; staged and
    polled exchange; tensor-core, CUDA-core and CSR projections) against the oracle."""
    scale = min(0.3, 2.0 / np.sqrt(c["H"] + c["in_dim"]))
    w = wl.Workload("fuzz", c["L"], c["bidir"], c["in_dim"], c["H"], c["T"], c["B"], c["dtype"], scale,
                    density=c["density"], seed=c["seed"])
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w) if c["states"] else (None, None)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got = run_gpu(w, weights, x, h0, c0, exec_mode=c["mode"])
    assert_close(got, ref, w.dtype, "fuzz")


def _fuzz_batched(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        H = int(rng.choice([rng.integers(8, 150), rng.integers(150, 700), rng.integers(700, 1700)]))
        cases.append(dict(L=int(rng.integers(1, 3)), bidir=bool(rng.integers(0, 2)), in_dim=int(rng.integers(1, 120)), H=H,
                          T=int(rng.integers(1, 6)), B=int(rng.integers(5, 33)), states=bool(rng.integers(0, 2)), seed=3000 + i))
    return cases


@pytest.mark.parametrize("c", _fuzz_batched(16, 77), ids=lambda c: "L{L}D{d}_in{in_dim}_H{H}_T{T}_B{B}".format(d=1 + c["bidir"], **c))
def test_random_batched_shapes(oracle, c):
    """Batches of 5 to 32 sequences at random widths: the batched tensor-core recurrence with and without
    cluster pairs (odd CTA counts, slices too tall for a pair), its fall-backs (slice too large), and wide
    bidirectional stacks whose directions run one after the other."""
    scale = min(0.3, 2.0 / np.sqrt(c["H"] + c["in_dim"]))
    w = wl.Workload("fuzzb", c["L"], c["bidir"], c["in_dim"], c["H"], c["T"], c["B"], "bf16", scale, seed=c["seed"])
    weights, x = wl.make(w)
    h0, c0 = wl.make_states(w) if c["states"] else (None, None)
    ref = oracle.forward(weights, x, h0, c0, layers=w.layers, bidir=w.bidir, hidden=w.hidden)
    got = run_gpu(w, weights, x, h0, c0)
    assert_close(got, ref, "bf16", "fuzz batched")


# ---------------------------------------------------------------- the step-cost probe
def test_probe_modes_run_to_the_end_and_the_whole_step_mode_is_exact(oracle):
    """lstm_probe selects measurement builds that leave parts of the recurrent step out.  Every mode must run to
    its end without a timeout (the exchange still completes: every unit publishes a word per step), the whole-step
    mode must give the normal results, and handles on other kernels must refuse a mask."""
    import torch
    import paper_1901_10997_b200 as pkg
    for mode, density in (("dense", 1.0), ("csr", 0.2)):
        w = small("probe", 2, False, 48, 300, 9, 1, "bf16", density=density, seed=55)
        weights, x = wl.make(w)
        ref = oracle.forward(weights, x, layers=2, bidir=False, hidden=300)
        m = pkg.LSTM(weights, layers=2, in_dim=48, hidden=300, dtype="bf16", exec_mode=mode, max_T=w.T, max_B=1)
        xd = torch.from_numpy(x).cuda()
        for mask in (pkg.LSTM_PROBE_NO_PRODUCTS, pkg.LSTM_PROBE_NO_GATES, pkg.LSTM_PROBE_NO_EXCHANGE,
                     pkg.LSTM_PROBE_NO_PRODUCTS | pkg.LSTM_PROBE_NO_GATES, pkg.LSTM_PROBE_NO_EXCHANGE | pkg.LSTM_PROBE_NO_GATES):
            if mode == "csr" and m.info()["layer_wavefront"]:
                break
            try:
                m.probe(mask)
            except pkg.LstmError as e:                     # a stack served by the wavefront kernel has no probe build
                assert e.code == pkg.LSTM_ERR_UNSUPPORTED
                break
            m.forward(xd)
            assert m.status() == pkg.LSTM_OK, (mode, mask)
        if m.info()["recur_register_resident"] or m.info()["recur_csr_register_resident"]:
            m.probe(pkg.LSTM_PROBE_WHOLE_STEP)
            y, hT, cT = m.forward(xd)
            m.check()
            assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"probe whole step {mode}")
        m.probe(0)
        y, hT, cT = m.forward(xd)
        m.check()
        assert_close((y.cpu().numpy(), hT.cpu().numpy(), cT.cpu().numpy()), ref, "bf16", f"after the probe {mode}")
        m.close()
    wf = small("probe_fp32", 1, False, 8, 20, 3, 1, "fp32", seed=56)
    weights, x = wl.make(wf)
    m = pkg.LSTM(weights, layers=1, in_dim=8, hidden=20, dtype="fp32", max_T=3, max_B=1)
    with pytest.raises(pkg.LstmError) as e:
        m.probe(pkg.LSTM_PROBE_NO_PRODUCTS)
    assert e.value.code == pkg.LSTM_ERR_UNSUPPORTED
    m.close()
