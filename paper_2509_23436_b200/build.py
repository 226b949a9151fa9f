"""Builds liblot.so (the CUDA library behind include/lot.h) in-tree with nvcc for sm_100a.

    python -m paper_2509_23436_b200.build [--force] [--verbose] [--debug]

--debug builds liblot_debug.so instead: the same sources with -DLOT_DEBUG (index checks in the general-path and
backward kernels that record a status flag and skip the access).  LOT_LIBRARY=<path> makes the binding load it.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "liblot.so")
LIB_DEBUG = os.path.join(PKG, "liblot_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-cudart", "static", "-diag-suppress", "128",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))


def build_lib(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    newest = max(os.path.getmtime(p) for p in _deps())
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-DLOT_DEBUG"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) + \
        ["-o", lib] + sources() + ["-lcuda"]
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build_lib(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
