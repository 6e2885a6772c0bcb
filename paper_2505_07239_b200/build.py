"""Build step of the CUDA library: one nvcc invocation for sm_100a, in-tree."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libcomet_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
]


def _sources():
    return sorted(os.path.join(_CSRC, f) for f in os.listdir(_CSRC) if f.endswith(".cu"))


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)]
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "comet.h"))
    return max(os.path.getmtime(p) for p in paths)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libcomet_b200.so next to this file (skipped when up to date)."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", LIB_PATH, *_sources()]
    subprocess.check_call(cmd)
    return LIB_PATH


if __name__ == "__main__":
    import sys

    print(build_library(force=True, verbose="-v" in sys.argv))
