"""Build ``libpsops.so`` (CUDA kernels + C ABI) for sm_100a with nvcc.

The library is built in-tree, next to this file.  nvcc cross-compiles without a
GPU, so this runs on any box with the CUDA toolkit.
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
SOURCES = [os.path.join(_HERE, "csrc", "psops.cu")]
HEADERS = [os.path.join(_ROOT, "include", "psops.h"), os.path.join(_HERE, "csrc", "psops_kernels.cuh")]
LIBRARY = os.path.join(_HERE, "libpsops.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo",
    "-fmad=false",              # no contraction the source does not spell out
    "-Xcompiler", "-fPIC", "-shared",
    "-I", os.path.join(_ROOT, "include"),
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIBRARY):
        return True
    built = os.path.getmtime(LIBRARY)
    return any(os.path.getmtime(f) > built for f in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources."""
    if not force and not is_stale():
        return LIBRARY
    tmp = LIBRARY + ".tmp.%d" % os.getpid()
    cmd = [_nvcc(), *NVCC_FLAGS, "-o", tmp, *SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
