import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, where no device is visible."""
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device visible")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


def pytest_sessionfinish(session, exitstatus):
    """With LSTM_B200_ERRLOG=<file>, writes every (case, tensor, storage type, floored, scaled) error the GPU
    parity helpers measured in this session, one JSON record per line."""
    path = os.environ.get("LSTM_B200_ERRLOG")
    if not path:
        return
    try:
        import json
        import gpu_util
        with open(path, "w") as f:
            for rec in gpu_util.ERR_LOG:
                f.write(json.dumps(rec) + "\n")
    except Exception:
        pass
