"""Builds ``libfastsgd_b200.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libfastsgd_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fno-fast-math",
    "--fmad=false", "--ftz=false", "--prec-div=true", "--prec-sqrt=true",
    "-cudart", "static",
]


def sources():
    return [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC)) if f.endswith(".cu")]


def _deps():
    out = [os.path.join(_ROOT, "include", "fastsgd.h")]
    out += [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)]
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library if it is missing or older than its sources.  With FASTSGD_TRACE=1 in the
    environment the kernels are built with their %globaltimer phase stamps (a profiling build: force it,
    and force a plain build afterwards)."""
    stale = (not os.path.exists(LIB_PATH)) or any(
        os.path.getmtime(d) > os.path.getmtime(LIB_PATH) for d in _deps())
    if force or stale:
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        trace = ["-DFASTSGD_TRACE"] if os.environ.get("FASTSGD_TRACE") == "1" else []
        cmd = [nvcc, *NVCC_FLAGS, *trace, *(["-Xptxas", "-v"] if verbose else []), "-o", LIB_PATH, *sources()]
        subprocess.check_call(cmd)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
