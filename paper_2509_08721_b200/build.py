"""Build the CUDA library in-tree with nvcc for sm_100a (no torch extension machinery:
the C ABI has no torch types)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsapo_b200.so")
LIB_CHECKED = os.path.join(HERE, "libsapo_b200_checked.so")     # the same sources with -DSAPO_BOUNDS_CHECK
LIB_STATS = os.path.join(HERE, "libsapo_b200_stats.so")         # ... with -DSAPO_WAIT_STATS (cycle counters)
SOURCES = ["runtime.cu", "pack.cu", "advantages.cu", "select.cu", "adam.cu", "lmhead.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "--shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "sapo.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False, stats: bool = False) -> str:
    """Build the library.  checked=True: the bounds-checking variant; stats=True: the variant whose
    GEMM kernels count their own cycles, nanoseconds and waits (read by bench.py); both are built
    beside the regular library and loaded through SAPO_B200_LIB."""
    lib = LIB_CHECKED if checked else (LIB_STATS if stats else LIB)
    if not force and not needs_build(lib):
        return lib
    extra = (["-DSAPO_BOUNDS_CHECK"] if checked else []) + (["-DSAPO_WAIT_STATS"] if stats else [])
    cmd = [_nvcc()] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checked="--checked" in sys.argv, stats="--stats" in sys.argv))
