"""The GPU parity suites once more under the bounds-checked build of the library (libhos_debug.so,
-DHOS_DEBUG_BOUNDS): every data-dependent index into shared or global memory is checked, a bad
one is counted and skipped.  The run must give the oracle's results AND count no violation."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_suites_under_the_bounds_checked_build():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    env = dict(os.environ, HOS_LIB_VARIANT="debug")
    cmd = [sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_gpu_random.py",
           "tests/test_gpu_stream.py", "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert "bounds violations: 0" in r.stdout, tail
