"""The checked build (liblstm_b200_checked.so: the same kernels compiled with index and shared-memory carve-up
checks that record LSTM_ERR_INTERNAL instead of trapping) runs the small-shape, tensor-core-edge, wavefront and
sparse parity cases.  A memory checker cannot be run on the test machines; this is its stand-in: every shape the
planner can emit for these cases must pass with the checks compiled in, and `m.check()` in every one of those
tests turns a recorded violation into a failure."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

SELECTION = ("test_small_shapes or test_batched_tensor_core_recurrence or test_masked_small or test_random_batched_shapes "
             "or test_wavefront_against_oracle or test_pruned_units_small or test_chunked_calls_carry_state "
             "or test_wide_bidirectional_stack or test_config2_b1_full or test_config4")


def test_parity_cases_pass_with_the_index_checks_compiled_in():
    from paper_1901_10997_b200 import build
    lib = build.LIB_CHECKED if build.LIB_CHECKED.exists() else build.build(checked=True)     # built with the normal library
    assert lib.exists()
    env = dict(os.environ, LSTM_B200_LIBRARY="checked")
    r = subprocess.run([sys.executable, "-m", "pytest", str(ROOT / "tests"), "-m", "gpu", "-q", "-x", "-k", SELECTION,
                        "--deselect", "tests/test_gpu_checked_build.py"], env=env, capture_output=True, text=True, timeout=1500, cwd=str(ROOT))
    tail = (r.stdout or "")[-1500:]
    assert r.returncode == 0, tail
    assert " passed" in tail and "failed" not in tail, tail
