"""The small-shape parity tests once more against the bounds-checking build of the library
(-DSAPO_BOUNDS_CHECK: every index a kernel computes before a global-memory access is compared
with the extent of its array, a violation is counted and the access left out).  This stands in
for a memory checker: the tests must pass as before and the kernels must count no violation.
The tests run in a child process because a process loads one build of the library."""
import os
import subprocess
import sys

import pytest

from paper_2509_08721_b200 import build

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FILES = ["tests/test_gpu_parity.py", "tests/test_gpu_fused.py", "tests/test_gpu_gather.py",
         "tests/test_gpu_bf16_outputs.py", "tests/test_gpu_contract.py", "tests/test_gpu_bwd_active.py"]


def test_small_shapes_pass_and_count_no_violation_in_the_checked_build(tmp_path):
    lib = build.build(checked=True)
    report = tmp_path / "violations.txt"
    env = dict(os.environ, SAPO_B200_LIB=lib, SAPO_BOUNDS_REPORT=str(report))
    res = subprocess.run([sys.executable, "-m", "pytest", *FILES, "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert report.read_text() == "0"


def test_the_regular_build_says_it_is_not_checked():
    from paper_2509_08721_b200 import binding as B
    if os.environ.get("SAPO_B200_LIB"):
        pytest.skip("another build of the library is loaded")
    assert B.load().sapo_debug_bounds_violations() == -1
