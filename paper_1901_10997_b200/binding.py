"""ctypes binding of include/lstm_b200.h: same names, argument marshalling only.

The module-level functions mirror the C entry points one to one (pointers as integers).  ``LSTM`` is
a convenience wrapper that takes numpy / torch arrays, keeps the handle, and allocates outputs with
torch (device memory and streams are the only things torch is used for).
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

LSTM_F32, LSTM_BF16W_F32S = 0, 1
LSTM_DENSE, LSTM_CSR = 0, 1
LSTM_OK, LSTM_ERR_INVALID, LSTM_ERR_UNSUPPORTED, LSTM_ERR_CUDA, LSTM_ERR_NOMEM, LSTM_ERR_TIMEOUT, LSTM_ERR_INTERNAL = range(7)
LSTM_K_STAGE, LSTM_K_PROJ, LSTM_K_RECUR, LSTM_K_COUNT = 0, 1, 2, 3
LSTM_PROBE_NO_PRODUCTS, LSTM_PROBE_NO_GATES, LSTM_PROBE_NO_EXCHANGE, LSTM_PROBE_WHOLE_STEP = 1, 2, 4, 8

import os as _os

# LSTM_B200_LIBRARY=checked loads the build with index checks compiled into the kernels (same ABI)
_LIB_PATH = Path(__file__).resolve().parent / ("liblstm_b200_checked.so" if _os.environ.get("LSTM_B200_LIBRARY") == "checked"
                                               else "liblstm_b200.so")
_lib = None


class LstmError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"lstm_b200 error {code}: {message}")
        self.code = code


class _Weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("wx", "wh", "b", "mask_x", "mask_h", "wx_rowptr", "wx_col", "wx_val",
                 "wh_rowptr", "wh_col", "wh_val")]


class _HWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("ux", "uh", "a", "w", "b", "mask_ux", "mask_uh", "mask_w")]


def lib_path() -> Path:
    return _LIB_PATH


def load_library():
    """Loads liblstm_b200.so (built by paper_1901_10997_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(
                f"{_LIB_PATH} not found: build it with `python -m paper_1901_10997_b200.build`; "
                "there is no fallback path")
        lib = ctypes.CDLL(str(_LIB_PATH))
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.lstm_create.restype = ci
        lib.lstm_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, vp, ci, ci, ci, vp]
        lib.hlstm_create.restype = ci
        lib.hlstm_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ci, vp, ci, ci, vp]
        lib.lstm_forward.restype = ci
        lib.lstm_forward.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, vp, vp]
        lib.lstm_input_projection.restype = ci
        lib.lstm_input_projection.argtypes = [vp, vp, ci, ci, vp, vp]
        lib.lstm_forward_host.restype = ci
        lib.lstm_forward_host.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, vp, vp]
        lib.lstm_status.restype = ci
        lib.lstm_status.argtypes = [vp]
        lib.lstm_destroy.restype = ci
        lib.lstm_destroy.argtypes = [vp]
        lib.lstm_last_error.restype = ctypes.c_char_p
        lib.lstm_last_error.argtypes = [vp]
        lib.lstm_profile_enable.restype = ci
        lib.lstm_profile_enable.argtypes = [vp, ci]
        lib.lstm_profile_read.restype = ci
        lib.lstm_profile_read.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ctypes.c_float)]
        lib.lstm_info.restype = ci
        lib.lstm_info.argtypes = [vp, ctypes.POINTER(ctypes.c_int64), ci]
        lib.lstm_selftest_timeout.restype = ci
        lib.lstm_selftest_timeout.argtypes = [vp, ci, ctypes.c_longlong]
        lib.lstm_probe.restype = ci
        lib.lstm_probe.argtypes = [vp, ci]
        lib.lstm_forward_noalloc.restype = ci
        lib.lstm_forward_noalloc.argtypes = [vp, vp, vp, ci, ci, vp, ci, ci, vp, vp, vp, vp, vp, vp, ctypes.c_char_p, ci]
        pi, pd, pf = ctypes.POINTER(ci), ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_float)
        lib.lstm_lhp_points.restype = ci
        lib.lstm_lhp_points.argtypes = [pi, pd, ci, ctypes.c_double, pi, pi]
        lib.lstm_nearest_lhp.restype = ci
        lib.lstm_nearest_lhp.argtypes = [pi, pd, ci, ctypes.c_double, ci, pi]
        lib.lstm_fold_input_affine.restype = ci
        lib.lstm_fold_input_affine.argtypes = [pf, pf, ci, ci, pf, pf, pf, pf]
        lib.lstm_csr_lane_layout.restype = ci
        lib.lstm_csr_lane_layout.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, pi, ctypes.POINTER(ctypes.c_longlong)]
        _lib = lib
    return _lib


# ---------------------------------------------------------------- one-to-one entry points
def lstm_last_error(handle=None) -> str:
    s = load_library().lstm_last_error(handle)
    return s.decode() if s else ""


def lstm_create(layers, in_dim, hidden, bidir, dtype, weights_ptr, exec_mode, max_T, max_B, stream=0):
    """Returns (code, handle).  ``weights_ptr``: address of an lstm_weights[layers*(1+bidir)] array."""
    out = ctypes.c_void_p()
    rc = load_library().lstm_create(ctypes.byref(out), layers, in_dim, hidden, int(bool(bidir)), dtype,
                                    weights_ptr, exec_mode, max_T, max_B, stream or None)
    return rc, out.value


def hlstm_create(layers, in_dim, hidden, gate_hidden, bidir, dtype, weights_ptr, max_T, max_B, stream=0):
    """Returns (code, handle).  ``weights_ptr``: address of an hlstm_weights[layers*(1+bidir)] array."""
    out = ctypes.c_void_p()
    rc = load_library().hlstm_create(ctypes.byref(out), layers, in_dim, hidden, gate_hidden, int(bool(bidir)), dtype,
                                     weights_ptr, max_T, max_B, stream or None)
    return rc, out.value


def lstm_forward(handle, x, T, B, h0, c0, y, hT, cT, stream=0):
    return load_library().lstm_forward(handle, x or None, T, B, h0 or None, c0 or None, y or None,
                                       hT or None, cT or None, stream or None)


def lstm_input_projection(handle, x, T, B, g, stream=0):
    return load_library().lstm_input_projection(handle, x or None, T, B, g or None, stream or None)


def lstm_forward_host(handle, x, T, B, h0, c0, y, hT, cT, stream=0):
    return load_library().lstm_forward_host(handle, x or None, T, B, h0 or None, c0 or None, y or None,
                                            hT or None, cT or None, stream or None)


def lstm_status(handle):
    return load_library().lstm_status(handle)


def lstm_destroy(handle):
    return load_library().lstm_destroy(handle)


def lstm_selftest_timeout(handle, cta, spin_limit=0):
    return load_library().lstm_selftest_timeout(handle, cta, spin_limit)


def lstm_probe(handle, parts_left_out):
    return load_library().lstm_probe(handle, int(parts_left_out))


def lstm_profile_enable(handle, on):
    return load_library().lstm_profile_enable(handle, int(bool(on)))


def lstm_profile_read(handle):
    n = (ctypes.c_int * LSTM_K_COUNT)()
    ms = (ctypes.c_float * LSTM_K_COUNT)()
    rc = load_library().lstm_profile_read(handle, n, ms)
    return rc, list(n), list(ms)


def lstm_info(handle):
    out = (ctypes.c_int64 * 32)()
    n = load_library().lstm_info(handle, out, 32)
    keys = ["sm_count", "ctas_per_dir", "threads", "smem_bytes", "rows_resident", "rows_streamed",
            "proj_splits", "proj_tensor_core", "launches_per_forward", "recur_register_resident",
            "col_tiles_in_registers", "col_tiles_in_smem", "recur_batched_tensor_core",
            "recur_csr_register_resident", "csr_slots_per_lane", "csr_bank_conflict_wavefronts",
            "compact_hidden", "units_removed", "layer_wavefront"]
    return {k: int(out[i]) for i, k in enumerate(keys[:n])}


def _curve(sizes, latency):
    n = len(sizes)
    if n != len(latency):
        raise ValueError("sizes and latency differ in length")
    return (ctypes.c_int * n)(*[int(v) for v in sizes]), (ctypes.c_double * n)(*[float(v) for v in latency]), n


def lstm_lhp_points(sizes, latency, eps=0.0):
    """Returns (code, flags, count): flags[i] = 1 where sizes[i] is a latency hysteresis point."""
    cs, cl, n = _curve(sizes, latency)
    flags = (ctypes.c_int * max(n, 1))()
    count = ctypes.c_int(0)
    rc = load_library().lstm_lhp_points(cs, cl, n, float(eps), flags, ctypes.byref(count))
    return rc, [int(flags[i]) for i in range(n)], int(count.value)


def lstm_nearest_lhp(sizes, latency, requested, eps=0.0):
    """Returns (code, size): the smallest latency hysteresis point >= requested."""
    cs, cl, n = _curve(sizes, latency)
    out = ctypes.c_int(0)
    rc = load_library().lstm_nearest_lhp(cs, cl, n, float(eps), int(requested), ctypes.byref(out))
    return rc, int(out.value)


def lstm_fold_input_affine(wx, b, scale, shift):
    """Returns (code, wx_folded, b_folded) as new float32 arrays; b, scale, shift may be None."""
    import numpy as np
    wx = np.ascontiguousarray(wx, dtype=np.float32)
    rows, cols = wx.shape
    as_f = lambda a, n: None if a is None else np.ascontiguousarray(a, dtype=np.float32).reshape(n)
    b, scale, shift = as_f(b, rows), as_f(scale, cols), as_f(shift, cols)
    wx_out, b_out = np.empty_like(wx), np.empty(rows, np.float32)
    pf = ctypes.POINTER(ctypes.c_float)
    ptr = lambda a: None if a is None else a.ctypes.data_as(pf)
    rc = load_library().lstm_fold_input_affine(ptr(wx), ptr(b), rows, cols, ptr(scale), ptr(shift), ptr(wx_out), ptr(b_out))
    return rc, wx_out, b_out


def lstm_csr_lane_layout(rowptr, col, val, hidden, ctas, warps, kspan, slots=None):
    """Returns (code, longest, rows, entries, conflict_wavefronts); with ``slots`` None only the list lengths and
    rows are computed (entries is None).  rows: uint32 [ctas, warps, 32]; entries: uint32 [ctas, warps, slots, 32]."""
    rowptr = np.ascontiguousarray(rowptr, np.int32)
    col = np.ascontiguousarray(col, np.int32)
    val = np.ascontiguousarray(val, np.float32)
    rows = np.zeros((ctas, warps, 32), np.uint32)
    longest = ctypes.c_int(0)
    conflicts = ctypes.c_longlong(0)
    entries = None if slots is None else np.zeros((ctas, warps, slots, 32), np.uint32)
    rc = load_library().lstm_csr_lane_layout(rowptr.ctypes.data, col.ctypes.data, val.ctypes.data, hidden, ctas, warps, kspan,
                                             0 if slots is None else slots, None if entries is None else entries.ctypes.data,
                                             rows.ctypes.data, ctypes.byref(longest), ctypes.byref(conflicts))
    return rc, int(longest.value), rows, entries, int(conflicts.value)


def lstm_forward_noalloc(wx, wh, b, in_dim, hidden, x, T, B, h0, c0, y, hT, cT, stream=0):
    """One fp32 layer straight from the caller's device buffers (addresses as integers), using only
    the scratch array built into the library: for callers that may not allocate device memory.
    Returns (code, message)."""
    err = ctypes.create_string_buffer(512)
    rc = load_library().lstm_forward_noalloc(wx or None, wh or None, b or None, in_dim, hidden, x or None, T, B,
                                             h0 or None, c0 or None, y or None, hT or None, cT or None,
                                             stream or None, err, len(err))
    return rc, err.value.decode()


# ---------------------------------------------------------------- convenience wrapper
def _addr(a, keep):
    """Address of a numpy array or torch tensor (host or device); None -> 0."""
    if a is None:
        return 0
    if isinstance(a, np.ndarray):
        keep.append(a)
        return a.ctypes.data
    keep.append(a)
    return a.data_ptr()


def _as_c(a, np_dtype):
    """Contiguous array of the wanted dtype; torch tensors are kept as they are if already right."""
    if a is None:
        return None
    if isinstance(a, np.ndarray) or not hasattr(a, "data_ptr"):
        return np.ascontiguousarray(a, dtype=np_dtype)
    import torch
    want = {np.float32: torch.float32, np.uint8: torch.uint8, np.int32: torch.int32}[np_dtype]
    return a.to(want).contiguous()


class LSTM:
    """Owns one library handle.  ``weights``: list of dicts per (layer, direction) with ``wx``,
    ``wh``, optional ``b``, ``mask_x``, ``mask_h``, or ``wx_csr`` / ``wh_csr`` = (rowptr, col, val);
    gate row blocks i, f, g, o."""

    def __init__(self, weights, *, layers, in_dim, hidden, bidir=False, dtype="bf16", exec_mode="dense",
                 max_T, max_B, stream=0):
        self.layers, self.in_dim, self.hidden = int(layers), int(in_dim), int(hidden)
        self.dirs = 2 if bidir else 1
        self.max_T, self.max_B = int(max_T), int(max_B)
        self._handle = None
        n = self.layers * self.dirs
        if len(weights) != n:
            raise ValueError(f"need {n} weight sets, got {len(weights)}")
        arr = (_Weights * n)()
        keep = []
        for i, w in enumerate(weights):
            s = arr[i]
            if w.get("wx_csr") is not None:
                rp, col, val = w["wx_csr"]
                s.wx_rowptr, s.wx_col, s.wx_val = (_addr(_as_c(rp, np.int32), keep), _addr(_as_c(col, np.int32), keep),
                                                   _addr(_as_c(val, np.float32), keep))
            else:
                s.wx = _addr(_as_c(w["wx"], np.float32), keep)
                s.mask_x = _addr(_as_c(w.get("mask_x"), np.uint8), keep)
            if w.get("wh_csr") is not None:
                rp, col, val = w["wh_csr"]
                s.wh_rowptr, s.wh_col, s.wh_val = (_addr(_as_c(rp, np.int32), keep), _addr(_as_c(col, np.int32), keep),
                                                   _addr(_as_c(val, np.float32), keep))
            else:
                s.wh = _addr(_as_c(w["wh"], np.float32), keep)
                s.mask_h = _addr(_as_c(w.get("mask_h"), np.uint8), keep)
            s.b = _addr(_as_c(w.get("b"), np.float32), keep)
        dt = {"fp32": LSTM_F32, "bf16": LSTM_BF16W_F32S}[dtype]
        em = {"dense": LSTM_DENSE, "csr": LSTM_CSR}[exec_mode]
        rc, handle = lstm_create(self.layers, self.in_dim, self.hidden, bidir, dt,
                                 ctypes.cast(arr, ctypes.c_void_p), em, self.max_T, self.max_B, stream)
        if rc != LSTM_OK:
            raise LstmError(rc, lstm_last_error(None))
        self._handle = handle

    # -- helpers
    def _check(self, rc):
        if rc != LSTM_OK:
            raise LstmError(rc, lstm_last_error(self._handle))

    @property
    def handle(self):
        return self._handle

    def forward(self, x, h0=None, c0=None, *, want_state=True, out=None, stream=None):
        """x: CUDA float32 tensor [T,B,in_dim]; returns (y, hT, cT) CUDA tensors (hT, cT None if
        ``want_state`` is False).  Enqueued on torch's current stream unless ``stream`` is given."""
        import torch
        if not (x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()):
            raise ValueError("x must be a contiguous CUDA float32 tensor")
        T, B, _ = x.shape
        st = torch.cuda.current_stream().cuda_stream if stream is None else stream
        if out is None:
            y = torch.empty((T, B, self.dirs * self.hidden), dtype=torch.float32, device=x.device)
            hT = cT = None
            if want_state:
                hT = torch.empty((self.layers * self.dirs, B, self.hidden), dtype=torch.float32, device=x.device)
                cT = torch.empty_like(hT)
        else:
            y, hT, cT = out
        for s in (h0, c0):
            if s is not None and not (s.is_cuda and s.dtype == torch.float32 and s.is_contiguous()):
                raise ValueError("h0/c0 must be contiguous CUDA float32 tensors")
        self._check(lstm_forward(self._handle, x.data_ptr(), T, B,
                                 h0.data_ptr() if h0 is not None else 0, c0.data_ptr() if c0 is not None else 0,
                                 y.data_ptr(), hT.data_ptr() if hT is not None else 0,
                                 cT.data_ptr() if cT is not None else 0, st))
        return y, hT, cT

    def input_projection(self, x, *, out=None, stream=None):
        """First layer's input projection alone: x CUDA float32 [T,B,in_dim] -> [T,B,D,4*Hg] (gate blocks i,f,g,o)."""
        import torch
        T, B, _ = x.shape
        hg = getattr(self, "gate_hidden", None) or self.hidden
        if out is None:
            out = torch.empty((T, B, self.dirs, 4 * hg), dtype=torch.float32, device=x.device)
        st = torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(lstm_input_projection(self._handle, x.data_ptr(), T, B, out.data_ptr(), st))
        return out

    def forward_host(self, x, h0=None, c0=None, *, y=None, hT=None, cT=None, stream=0):
        """Host-buffer call: numpy arrays or CPU (ideally pinned) torch tensors in and out."""
        T, B, _ = x.shape
        keep = []
        if y is None:
            y = np.empty((T, B, self.dirs * self.hidden), np.float32)
            hT = np.empty((self.layers * self.dirs, B, self.hidden), np.float32)
            cT = np.empty_like(hT)
        self._check(lstm_forward_host(self._handle, _addr(x, keep), T, B, _addr(h0, keep), _addr(c0, keep),
                                      _addr(y, keep), _addr(hT, keep), _addr(cT, keep), stream))
        return y, hT, cT

    def status(self):
        return lstm_status(self._handle)

    def check(self):
        self._check(lstm_status(self._handle))

    def info(self):
        return lstm_info(self._handle)

    def selftest_timeout(self, cta, spin_limit=0):
        self._check(lstm_selftest_timeout(self._handle, cta, spin_limit))

    def probe(self, parts_left_out=0):
        """Step-cost measurement: leave parts of the recurrent step out (outputs undefined until reset to 0)."""
        self._check(lstm_probe(self._handle, parts_left_out))

    def profile_enable(self, on=True):
        self._check(lstm_profile_enable(self._handle, on))

    def profile_read(self):
        rc, n, ms = lstm_profile_read(self._handle)
        self._check(rc)
        return n, ms

    def close(self):
        if self._handle:
            lstm_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class HLSTM(LSTM):
    """H-LSTM cell (one ReLU hidden layer of width ``gate_hidden`` inside each gate).  ``weights``: list of
    dicts per (layer, direction) with ``ux`` [4Hh,in_l], ``uh`` [4Hh,H], ``w`` [4H,Hh], optional ``a``, ``b`` and
    keep-masks ``mask_ux``, ``mask_uh``, ``mask_w`` (uint8, same shapes);
    gate blocks i, f, g, o.  Forward, status and the other methods are those of ``LSTM``."""

    def __init__(self, weights, *, layers, in_dim, hidden, gate_hidden, bidir=False, dtype="bf16", max_T, max_B, stream=0):
        self.layers, self.in_dim, self.hidden = int(layers), int(in_dim), int(hidden)
        self.gate_hidden = int(gate_hidden)
        self.dirs = 2 if bidir else 1
        self.max_T, self.max_B = int(max_T), int(max_B)
        self._handle = None
        n = self.layers * self.dirs
        if len(weights) != n:
            raise ValueError(f"need {n} weight sets, got {len(weights)}")
        arr = (_HWeights * n)()
        keep = []
        for i, w in enumerate(weights):
            s = arr[i]
            s.ux = _addr(_as_c(w["ux"], np.float32), keep)
            s.uh = _addr(_as_c(w["uh"], np.float32), keep)
            s.w = _addr(_as_c(w["w"], np.float32), keep)
            s.a = _addr(_as_c(w.get("a"), np.float32), keep)
            s.b = _addr(_as_c(w.get("b"), np.float32), keep)
            for name in ("mask_ux", "mask_uh", "mask_w"):
                setattr(s, name, _addr(_as_c(w.get(name), np.uint8), keep))
        dt = {"fp32": LSTM_F32, "bf16": LSTM_BF16W_F32S}[dtype]
        rc, handle = hlstm_create(self.layers, self.in_dim, self.hidden, self.gate_hidden, bidir, dt,
                                  ctypes.cast(arr, ctypes.c_void_p), self.max_T, self.max_B, stream)
        if rc != LSTM_OK:
            raise LstmError(rc, lstm_last_error(None))
        self._handle = handle
