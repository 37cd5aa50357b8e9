"""Seeded synthetic workloads shared by the tests, the benchmark and the smoke check.

This module holds no LSTM arithmetic: it only draws weights, masks and inputs with the shapes and
value ranges of the paper's workloads (Section 5.1: Penn-Treebank language model, two stacked layers
of width 1500, sequence length 35/70; Section 5.2: DeepSpeech2-style stack of five bidirectional
layers of width 800), rounds them to the storage type once, and defines the error metric used to
compare two results.  The real datasets are not needed: only shapes and ranges are taken.

Recipe.  ``numpy.random.Generator(PCG64(seed))``; draw order: for each layer, for each direction:
``wx``, ``wh``, ``b`` (uniform in [-a, a]), then, for pruned workloads, ``mask_x``, ``mask_h``
(Bernoulli keep-masks, Section 4 "mask-based approach"; survivors are the dense draw times the mask);
finally ``x`` ~ N(0,1) of shape [T, B, in_dim].  Draws are float64, cast to float32 and, for the
bf16 storage type, rounded to nearest-even bf16 and widened back, so that every consumer receives
bit-identical values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np

SEED_BASE = 190110997 * 10


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    bidir: bool
    in_dim: int
    hidden: int
    T: int
    B: int
    dtype: str          # "fp32" | "bf16" (bf16 weights, fp32 state)
    scale: float        # weights and biases ~ U(-scale, scale)
    density: float = 1.0  # keep probability of the Bernoulli masks (1.0 = dense, no masks)
    seed: int = 0

    @property
    def dirs(self) -> int:
        return 2 if self.bidir else 1

    def in_l(self, layer: int) -> int:
        return self.in_dim if layer == 0 else self.dirs * self.hidden

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _seed(config_index: int, sub: int = 0) -> int:
    return (SEED_BASE + config_index) * 100003 + sub


def config1() -> Workload:
    """Small language-model shape: 2 layers, 200 -> 200, T=35, batch 20, fp32."""
    return Workload("cfg1_small_fp32", 2, False, 200, 200, 35, 20, "fp32", 0.1, seed=_seed(1))


def config2(B: int = 1) -> Workload:
    """Large language-model shape (two layers of width 1500), T=35, batch 1 or 20, bf16 weights."""
    return Workload(f"cfg2_ptb_large_B{B}", 2, False, 1500, 1500, 35, B, "bf16", 0.04,
                    seed=_seed(2))


def config3(H: int) -> Workload:
    """One point of the hidden-size sweep: 1 layer, input = hidden = H, T=35, batch 1, bf16."""
    return Workload(f"cfg3_sweep_H{H}", 1, False, H, H, 35, 1, "bf16", 1.0 / math.sqrt(H),
                    seed=_seed(3, H))


def config3_sizes():
    return list(range(128, 2048 + 1, 8))


def config4(density: float) -> Workload:
    """Pruned large language-model shape: Bernoulli keep-masks on wx and wh, survivors U(-0.1,0.1)."""
    return Workload(f"cfg4_pruned_d{density:g}", 2, False, 1500, 1500, 35, 1, "bf16", 0.1,
                    density=density, seed=_seed(4, int(round(density * 1000))))


def config5(B: int = 1) -> Workload:
    """Speech-model shape: 5 bidirectional layers, 1312 -> 800 (then 1600 -> 800), T=400."""
    return Workload(f"cfg5_ds2_B{B}", 5, True, 1312, 800, 400, B, "bf16", 0.035, seed=_seed(5))


def config5_width(H: int, B: int = 16) -> Workload:
    """The speech-model shape at another hidden width (the width sweep of the paper's Figure 3): 5
    bidirectional layers, 1312 -> H, then 2H -> H, T=400."""
    return Workload(f"ds2_sweep_H{H}_B{B}", 5, True, 1312, H, 400, B, "bf16", 1.0 / math.sqrt(H), seed=_seed(5, H))


def config2_units_pruned(B: int = 1) -> Workload:
    """Large language-model shape after row/column pruning (paper, Section 4.2 and Table 1 step (b): hidden
    width 1500 pruned to 1197): the same two layers of width 1500, with 303 hidden units per layer whose rows
    and columns are zero (see ``prune_units``)."""
    return Workload(f"cfg2_units_pruned_B{B}", 2, False, 1500, 1500, 35, B, "bf16", 0.04, seed=_seed(2, 1197))


def prune_units(w: Workload, weights, keep: int, seed_offset: int = 11):
    """Row/column pruning at the level of whole hidden units, the structure Algorithm 1 of the paper leaves
    behind: for every (layer, direction) a seeded random set of ``hidden - keep`` units loses all its incoming
    weights (the four gate rows of ``wx`` and ``wh``) and all its outgoing ones (its column of ``wh`` and of the
    next layer's ``wx``).  Biases stay.  Returns (weights with the zeros written in, removed) where
    ``removed[layer * dirs + d]`` is the sorted array of pruned units.  No arithmetic of the model happens here."""
    rng = np.random.Generator(np.random.PCG64(w.seed + seed_offset))
    H, D = w.hidden, w.dirs
    out = [{k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in e.items()} for e in weights]
    removed = []
    for l in range(w.layers):
        for d in range(D):
            gone = np.sort(rng.choice(H, size=H - keep, replace=False))
            removed.append(gone)
            e = out[l * D + d]
            rows = (np.arange(4)[:, None] * H + gone[None, :]).ravel()
            e["wx"][rows, :] = 0.0
            e["wh"][rows, :] = 0.0
            e["wh"][:, gone] = 0.0
            if l + 1 < w.layers:
                for d2 in range(D):
                    out[(l + 1) * D + d2]["wx"][:, d * H + gone] = 0.0
    for e in out:
        for m, name in (("mask_x", "wx"), ("mask_h", "wh")):
            if m in e:
                e[m] = (e[m].astype(bool) & (e[name] != 0)).astype(np.uint8)
    return out, removed


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 -> nearest-even bfloat16 -> float32 (finite inputs)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def make(w: Workload):
    """Draw one workload.  Returns (weights, x): ``weights`` is a list with one dict per
    (layer, direction) -- index layer*dirs + direction, direction 1 = reverse -- holding float32
    ``wx`` [4H,in_l], ``wh`` [4H,H], ``b`` [4H] (gate row blocks i,f,g,o) and, when density < 1,
    uint8 ``mask_x``, ``mask_h`` (the weight arrays already carry the zeros); ``x`` is float32
    [T,B,in_dim].
    """
    rng = np.random.Generator(np.random.PCG64(w.seed))
    store = round_to_bf16 if w.dtype == "bf16" else (lambda a: a)
    H = w.hidden
    weights = []
    for l in range(w.layers):
        for _d in range(w.dirs):
            in_l = w.in_l(l)
            wx = store(rng.uniform(-w.scale, w.scale, size=(4 * H, in_l)).astype(np.float32))
            wh = store(rng.uniform(-w.scale, w.scale, size=(4 * H, H)).astype(np.float32))
            b = store(rng.uniform(-w.scale, w.scale, size=(4 * H,)).astype(np.float32))
            entry = {"wx": wx, "wh": wh, "b": b}
            if w.density < 1.0:
                mx = (rng.random(size=(4 * H, in_l)) < w.density).astype(np.uint8)
                mh = (rng.random(size=(4 * H, H)) < w.density).astype(np.uint8)
                entry["wx"] = wx * mx
                entry["wh"] = wh * mh
                entry["mask_x"] = mx
                entry["mask_h"] = mh
            weights.append(entry)
    x = rng.standard_normal(size=(w.T, w.B, w.in_dim)).astype(np.float32)
    return weights, x


def make_hlstm(w: Workload, gate_hidden: int):
    """Weights of the H-LSTM cell (one hidden layer of width ``gate_hidden`` inside each gate) with the
    shape of workload ``w``: per (layer, direction) ``ux`` [4Hh,in_l], ``uh`` [4Hh,H], ``a`` [4Hh],
    ``w`` [4H,Hh], ``b`` [4H], all ~ U(-scale, scale), rounded to the storage type; then ``x``."""
    rng = np.random.Generator(np.random.PCG64(w.seed + 991))
    store = round_to_bf16 if w.dtype == "bf16" else (lambda a: a)
    H, Hh = w.hidden, gate_hidden
    weights = []
    for l in range(w.layers):
        for _d in range(w.dirs):
            in_l = w.in_l(l)
            weights.append({
                "ux": store(rng.uniform(-w.scale, w.scale, size=(4 * Hh, in_l)).astype(np.float32)),
                "uh": store(rng.uniform(-w.scale, w.scale, size=(4 * Hh, H)).astype(np.float32)),
                "a": store(rng.uniform(-w.scale, w.scale, size=(4 * Hh,)).astype(np.float32)),
                "w": store(rng.uniform(-w.scale, w.scale, size=(4 * H, Hh)).astype(np.float32)),
                "b": store(rng.uniform(-w.scale, w.scale, size=(4 * H,)).astype(np.float32)),
            })
    x = rng.standard_normal(size=(w.T, w.B, w.in_dim)).astype(np.float32)
    return weights, x


def make_states(w: Workload, seed_offset: int = 7):
    """Non-zero initial states h0 in (-1,1), c0 ~ N(0,0.5), float32 [L*D,B,H]."""
    rng = np.random.Generator(np.random.PCG64(w.seed + seed_offset))
    shape = (w.layers * w.dirs, w.B, w.hidden)
    h0 = rng.uniform(-0.9, 0.9, size=shape).astype(np.float32)
    c0 = (0.5 * rng.standard_normal(size=shape)).astype(np.float32)
    return h0, c0


TOLERANCE = {"fp32": 1e-4, "bf16": 2e-2}
FLOOR_FRACTION = 1e-3


def rel_err(got: np.ndarray, ref: np.ndarray):
    """Error of ``got`` against ``ref`` for one output tensor.

    Returns (floored, scaled):
      floored = max_i |got_i - ref_i| / max(|ref_i|, tau),  tau = 1e-3 * max_j |ref_j|
      scaled  = max_i |got_i - ref_i| / max_j |ref_j|
    Element-wise relative error is undefined where the reference crosses zero, so elements within
    0.1% of zero (relative to the tensor's largest magnitude) are judged against the floor.
    An all-zero reference is judged on absolute error.
    """
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if got.shape != ref.shape:
        raise ValueError(f"shape mismatch {got.shape} vs {ref.shape}")
    if ref.size == 0:
        return 0.0, 0.0
    if not np.all(np.isfinite(got)):
        return float("inf"), float("inf")
    diff = np.abs(got - ref)
    big = float(np.max(np.abs(ref)))
    if big == 0.0:
        m = float(np.max(diff))
        return m, m
    tau = FLOOR_FRACTION * big
    floored = float(np.max(diff / np.maximum(np.abs(ref), tau)))
    return floored, float(np.max(diff) / big)
