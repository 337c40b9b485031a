"""Builds the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libdistrl_b200.so")
# The checked build: every computed index is range-checked (DISTRL_BOUNDS_CHECK) and the pipelined scan runs
# with tiles of half the size (4 items per thread), so the same inputs are cut into tiles differently.
CHECKED_LIB_PATH = os.path.join(_PKG, "libdistrl_b200_checked.so")
CHECKED_FLAGS = ["-DDISTRL_BOUNDS_CHECK", "-DDISTRL_PIPE_ITEMS=4"]
SOURCES = ["api.cu", "retrace.cu", "priority.cu", "sampler.cu", "batch.cu", "replay.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every .cu under csrc/ into libdistrl_b200.so (no GPU needed); checked=True: the checked build."""
    out = CHECKED_LIB_PATH if checked else LIB_PATH
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest_source_mtime():
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-t", "0", "-I", INCLUDE, "-I", CSRC, "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += CHECKED_FLAGS if checked else os.environ.get("DISTRL_NVCC_EXTRA", "").split()   # e.g. -D overrides of tuning constants
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
