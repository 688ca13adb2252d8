import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """A run against the bounds-checking build of the library (see test_gpu_bounds_checked.py)
    leaves the number of violations its kernels counted in the file SAPO_BOUNDS_REPORT names."""
    path = os.environ.get("SAPO_BOUNDS_REPORT")
    if not path:
        return
    from paper_2509_08721_b200 import binding as B
    with open(path, "w") as f:
        f.write(str(int(B.load().sapo_debug_bounds_violations())))
