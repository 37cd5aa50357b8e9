"""The C-ABI library loads and exports every symbol include/lstm_b200.h declares (no GPU needed)."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_1901_10997_b200 import build
    path = build.build()
    return ctypes.CDLL(str(path))


def declared_functions():
    text = (ROOT / "include" / "lstm_b200.h").read_text()
    return sorted(set(re.findall(r"LSTM_API\s+[\w\s\*]+?\b(lstm_\w+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("lstm_create", "lstm_forward", "lstm_destroy", "lstm_forward_host", "lstm_last_error"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_names_match_header():
    import paper_1901_10997_b200 as pkg
    for name in declared_functions():
        assert callable(getattr(pkg, name)), name


def test_create_fails_loudly_without_device():
    """Without a usable device the library reports an error instead of computing anywhere else."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    import numpy as np
    import paper_1901_10997_b200 as pkg
    w = [{"wx": np.zeros((8, 3), np.float32), "wh": np.zeros((8, 2), np.float32)}]
    with pytest.raises(pkg.LstmError) as e:
        pkg.LSTM(w, layers=1, in_dim=3, hidden=2, dtype="fp32", max_T=2, max_B=1)
    assert e.value.code == pkg.LSTM_ERR_CUDA


def test_create_rejects_bad_arguments_before_touching_the_device():
    import paper_1901_10997_b200 as pkg
    rc, handle = pkg.lstm_create(0, 3, 2, 0, pkg.LSTM_F32, 0, pkg.LSTM_DENSE, 1, 1)
    assert rc == pkg.LSTM_ERR_INVALID and not handle
    assert "bad argument" in pkg.lstm_last_error(None)
    rc, _ = pkg.lstm_create(1, 3, 70000, 0, pkg.LSTM_F32, 1, pkg.LSTM_DENSE, 1, 1)
    assert rc == pkg.LSTM_ERR_UNSUPPORTED


def test_checked_build_exports_the_same_boundary():
    """liblstm_b200_checked.so (index checks compiled into the kernels) has the ABI of the normal build."""
    from paper_1901_10997_b200 import build
    lib = ctypes.CDLL(str(build.build(checked=True)))
    for name in declared_functions():
        assert hasattr(lib, name), name
