"""Build step of the CUDA library: one nvcc invocation for sm_100a, in-tree."""
from __future__ import annotations

import hashlib
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


STAMP_PATH = LIB_PATH + ".stamp"


def source_digest() -> str:
    """Hash of everything the library is built from (sources, the public header, the flags)."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    paths = sorted(os.path.join(_CSRC, f) for f in os.listdir(_CSRC))
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "comet.h"))
    for path in paths:
        with open(path, "rb") as fh:
            h.update(os.path.basename(path).encode())
            h.update(fh.read())
    return h.hexdigest()


def is_current() -> bool:
    """True when libcomet_b200.so exists and was built from the sources as they are now."""
    if not (os.path.exists(LIB_PATH) and os.path.exists(STAMP_PATH)):
        return False
    with open(STAMP_PATH) as fh:
        return fh.read().strip() == source_digest()


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libcomet_b200.so next to this file (skipped when the
    stamp written by the last build matches the current sources)."""
    if not force and is_current():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", LIB_PATH, *_sources()]
    subprocess.check_call(cmd)
    with open(STAMP_PATH, "w") as fh:
        fh.write(source_digest() + "\n")
    return LIB_PATH


if __name__ == "__main__":
    import sys

    print(build_library(force=True, verbose="-v" in sys.argv))
