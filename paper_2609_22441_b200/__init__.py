"""B200-native sorted-search edge-feature join (C ABI in include/ccr.h, CUDA kernels in csrc/).

Submodules, imported on first use: `binding` mirrors the C entry points (ctypes), `workloads` draws the
seeded synthetic inputs, `build` compiles the library in-tree for sm_100a.
"""
import importlib

__all__ = ["build", "workloads", "binding"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
