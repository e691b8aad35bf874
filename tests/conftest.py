import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_sessionfinish(session, exitstatus):
    """With the bounds-checked library (HOS_LIB_VARIANT=debug) a run only passes if no kernel
    indexed outside its tables."""
    if os.environ.get("HOS_LIB_VARIANT", "") != "debug":
        return
    try:
        import torch
        if not torch.cuda.is_available():
            return
        import paper_2502_15763_b200 as hos
        count, first = hos.hos_debug_bounds_violations()
    except Exception as exc:                       # the library could not be loaded: that is a failure too
        print(f"\nbounds check: could not read the violation count: {exc}")
        session.exitstatus = 1
        return
    print(f"\nbounds violations: {count}" + (f" (first: site {first[0]}, index {first[1]}, limit {first[2]})" if count else ""))
    if count != 0:
        session.exitstatus = 1
