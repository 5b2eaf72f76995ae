"""Builds the CUDA library in-tree: nvcc, sm_100a only, one shared object next to this file."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libccr.so")
SOURCES = [os.path.join(CSRC, "ccr_api.cu")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--shared", "-Xcompiler", "-fPIC",
]


def _deps():
    out = list(SOURCES)
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cuh", ".h", ".cu")):
                out.append(os.path.join(root, f))
    return out


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in _deps())


DEBUG_LIB = os.path.join(HERE, "libccr_debug.so")


def build_debug(force: bool = False) -> str:
    """The bounds-checked build (-DCCR_DEBUG_BOUNDS): every global address of the join kernels is checked against the
    launch's buffers; load it through CCR_LIB_OVERRIDE.  For tests, not for serving."""
    if not force and os.path.exists(DEBUG_LIB) and all(os.path.getmtime(p) <= os.path.getmtime(DEBUG_LIB) for p in _deps()):
        return DEBUG_LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = DEBUG_LIB + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc] + NVCC_FLAGS + ["-DCCR_DEBUG_BOUNDS", "-o", tmp] + SOURCES, check=True)
    os.replace(tmp, DEBUG_LIB)
    return DEBUG_LIB


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    if "--debug-bounds" in sys.argv:
        print(build_debug(force="--force" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
