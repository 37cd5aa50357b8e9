"""ctypes front end of ``lstm_oracle.c`` (test infrastructure only; see that file's header).

``forward`` runs the whole stack in double precision.  Each (layer, direction) is described by a
dict with ``wx`` [4H,in_l], ``wh`` [4H,H], optional ``b`` [4H], optional ``mask_x`` / ``mask_h``
(uint8, 1 = keep), or -- for the CSR walk -- ``wx_csr`` / ``wh_csr`` = (rowptr, col, val).
Gate rows are packed i, f, g, o (Section 4 cell equations with zero hidden layers per gate).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lstm_oracle.c"
_LIB = _HERE / "liblstm_oracle.so"
_lib = None


class _Weights(ctypes.Structure):
    _fields_ = [
        ("wx", ctypes.c_void_p), ("wh", ctypes.c_void_p), ("b", ctypes.c_void_p),
        ("mask_x", ctypes.c_void_p), ("mask_h", ctypes.c_void_p),
        ("wx_rowptr", ctypes.c_void_p), ("wx_col", ctypes.c_void_p), ("wx_val", ctypes.c_void_p),
        ("wh_rowptr", ctypes.c_void_p), ("wh_col", ctypes.c_void_p), ("wh_val", ctypes.c_void_p),
    ]


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (no fast-math, no contraction) into this directory."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        lib.lstm_oracle_forward.restype = ctypes.c_int
        lib.lstm_oracle_forward.argtypes = [ctypes.c_int] * 6 + [ctypes.c_void_p] * 7
        lib.hlstm_oracle_forward.restype = ctypes.c_int
        lib.hlstm_oracle_forward.argtypes = [ctypes.c_int] * 7 + [ctypes.c_void_p] * 7
        lib.lstm_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


class _HWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("ux", "uh", "a", "w", "b")]


def forward_hlstm(weights, x, h0=None, c0=None, *, layers: int, bidir: bool, hidden: int, gate_hidden: int):
    """H-LSTM stack (one ReLU hidden layer of width ``gate_hidden`` inside each gate; Section 4 with
    H* = one layer).  Each (layer, direction) dict holds ``ux`` [4Hh,in_l], ``uh`` [4Hh,H], ``w`` [4H,Hh]
    and optional ``a`` [4Hh], ``b`` [4H]; gate blocks i, f, g, o.  Returns (y, hT, cT) as float64."""
    lib = _load()
    L, D, H, Hh = int(layers), (2 if bidir else 1), int(hidden), int(gate_hidden)
    x = np.ascontiguousarray(x, dtype=np.float64)
    T, B, in_dim = x.shape
    if len(weights) != L * D:
        raise ValueError("need one weight set per (layer, direction)")
    keep = []

    def f32(a, shape):
        a = np.ascontiguousarray(a, dtype=np.float32)
        if a.shape != shape:
            raise ValueError(f"bad shape {a.shape}, expected {shape}")
        keep.append(a)
        return a

    arr = (_HWeights * (L * D))()
    for l in range(L):
        in_l = in_dim if l == 0 else D * H
        for d in range(D):
            w, s = weights[l * D + d], arr[l * D + d]
            s.ux = _ptr(f32(w["ux"], (4 * Hh, in_l)))
            s.uh = _ptr(f32(w["uh"], (4 * Hh, H)))
            s.w = _ptr(f32(w["w"], (4 * H, Hh)))
            if w.get("a") is not None:
                s.a = _ptr(f32(w["a"], (4 * Hh,)))
            if w.get("b") is not None:
                s.b = _ptr(f32(w["b"], (4 * H,)))

    def state(a):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=np.float64)
        if a.shape != (L * D, B, H):
            raise ValueError(f"bad state shape {a.shape}")
        keep.append(a)
        return a

    h0, c0 = state(h0), state(c0)
    y = np.zeros((T, B, D * H), dtype=np.float64)
    hT = np.zeros((L * D, B, H), dtype=np.float64)
    cT = np.zeros((L * D, B, H), dtype=np.float64)
    rc = lib.hlstm_oracle_forward(L, D, in_dim, H, Hh, T, B, ctypes.cast(arr, ctypes.c_void_p),
                                  _ptr(x), _ptr(h0), _ptr(c0), _ptr(y), _ptr(hT), _ptr(cT))
    if rc != 0:
        raise RuntimeError(f"hlstm_oracle_forward failed with code {rc}")
    return y, hT, cT


def input_projection(weights, x, *, bidir: bool, hidden: int):
    """The input half of the first layer's gate pre-activations for every position, written out as its
    definition in float64 (Section 4: the x_t part of W [x_t, h_{t-1}] + b):
    g[t,b,d,q*H+j] = b_q[j] + sum_k (Wx (x) Msk)[q*H+j,k] x[t,b,k].  ``weights``: the first layer's dict
    per direction (``wx``, optional ``b``, ``mask_x``, or ``wx_csr``).  Returns [T,B,D,4H] float64."""
    x = np.asarray(x, dtype=np.float64)
    T, B, in_dim = x.shape
    D, H = (2 if bidir else 1), int(hidden)
    g = np.zeros((T, B, D, 4 * H), dtype=np.float64)
    for d in range(D):
        w = weights[d]
        if w.get("wx_csr") is not None:
            rp, col, val = w["wx_csr"]
            wx = np.zeros((4 * H, in_dim), dtype=np.float64)
            for r in range(4 * H):
                wx[r, np.asarray(col[rp[r]:rp[r + 1]])] = np.asarray(val[rp[r]:rp[r + 1]], dtype=np.float64)
        else:
            wx = np.asarray(w["wx"], dtype=np.float64)
            if w.get("mask_x") is not None:
                wx = wx * (np.asarray(w["mask_x"]) != 0)
        if wx.shape != (4 * H, in_dim):
            raise ValueError(f"bad wx shape {wx.shape}")
        bias = np.asarray(w["b"], dtype=np.float64) if w.get("b") is not None else np.zeros(4 * H)
        g[:, :, d, :] = x @ wx.T + bias
    return g


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().lstm_oracle_threads())


def dense_to_csr(w: np.ndarray, mask: np.ndarray | None = None):
    """(rowptr int32, col int32, val float32) of the kept entries of ``w`` in row-major order.

    With a mask, exactly the masked-in positions are kept (even if the value there is 0.0);
    without one, the nonzero entries are kept.
    """
    w = np.asarray(w, dtype=np.float32)
    keep = (np.asarray(mask) != 0) if mask is not None else (w != 0)
    counts = keep.sum(axis=1)
    rowptr = np.zeros(w.shape[0] + 1, dtype=np.int32)
    np.cumsum(counts, out=rowptr[1:])
    _, cols = np.nonzero(keep)
    return rowptr, cols.astype(np.int32), np.ascontiguousarray(w[keep], dtype=np.float32)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def forward(weights, x, h0=None, c0=None, *, layers: int, bidir: bool, hidden: int):
    """Run the stack; returns (y [T,B,D*H], hT [L*D,B,H], cT [L*D,B,H]) as float64 arrays."""
    lib = _load()
    L, D, H = int(layers), (2 if bidir else 1), int(hidden)
    x = np.ascontiguousarray(x, dtype=np.float64)
    T, B, in_dim = x.shape
    if len(weights) != L * D:
        raise ValueError("need one weight set per (layer, direction)")
    keep = []          # keeps converted arrays alive for the duration of the call

    def f32(a, shape):
        a = np.ascontiguousarray(a, dtype=np.float32)
        if a.shape != shape:
            raise ValueError(f"bad shape {a.shape}, expected {shape}")
        keep.append(a)
        return a

    def u8(a, shape):
        a = np.ascontiguousarray(a, dtype=np.uint8)
        if a.shape != shape:
            raise ValueError(f"bad mask shape {a.shape}, expected {shape}")
        keep.append(a)
        return a

    def csr(t, nrow, ncol):
        rp, col, val = t
        rp = np.ascontiguousarray(rp, dtype=np.int32)
        col = np.ascontiguousarray(col, dtype=np.int32)
        val = np.ascontiguousarray(val, dtype=np.float32)
        if rp.shape != (nrow + 1,) or rp[0] != 0 or rp[-1] != col.size or col.size != val.size:
            raise ValueError("malformed CSR")
        if col.size and (col.min() < 0 or col.max() >= ncol or np.any(np.diff(rp) < 0)):
            raise ValueError("malformed CSR")
        keep.extend([rp, col, val])
        return rp, col, val

    arr = (_Weights * (L * D))()
    for l in range(L):
        in_l = in_dim if l == 0 else D * H
        for d in range(D):
            w = weights[l * D + d]
            s = arr[l * D + d]
            if w.get("wx_csr") is not None:
                rp, col, val = csr(w["wx_csr"], 4 * H, in_l)
                s.wx_rowptr, s.wx_col, s.wx_val = _ptr(rp), _ptr(col), _ptr(val)
            else:
                s.wx = _ptr(f32(w["wx"], (4 * H, in_l)))
                if w.get("mask_x") is not None:
                    s.mask_x = _ptr(u8(w["mask_x"], (4 * H, in_l)))
            if w.get("wh_csr") is not None:
                rp, col, val = csr(w["wh_csr"], 4 * H, H)
                s.wh_rowptr, s.wh_col, s.wh_val = _ptr(rp), _ptr(col), _ptr(val)
            else:
                s.wh = _ptr(f32(w["wh"], (4 * H, H)))
                if w.get("mask_h") is not None:
                    s.mask_h = _ptr(u8(w["mask_h"], (4 * H, H)))
            if w.get("b") is not None:
                s.b = _ptr(f32(w["b"], (4 * H,)))

    def state(a):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=np.float64)
        if a.shape != (L * D, B, H):
            raise ValueError(f"bad state shape {a.shape}")
        keep.append(a)
        return a

    h0, c0 = state(h0), state(c0)
    y = np.zeros((T, B, D * H), dtype=np.float64)
    hT = np.zeros((L * D, B, H), dtype=np.float64)
    cT = np.zeros((L * D, B, H), dtype=np.float64)
    rc = lib.lstm_oracle_forward(L, D, in_dim, H, T, B, ctypes.cast(arr, ctypes.c_void_p),
                                 _ptr(x), _ptr(h0), _ptr(c0), _ptr(y), _ptr(hT), _ptr(cT))
    if rc != 0:
        raise RuntimeError(f"lstm_oracle_forward failed with code {rc}")
    return y, hT, cT
