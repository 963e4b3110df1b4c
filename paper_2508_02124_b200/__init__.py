"""B200-native (sm_100a) hot path of Dynamic Mask Attention: mask build, fused forward, fused backward.

The kernels live in ``csrc/`` behind a C-ABI shared library (``include/dma.h``); ``binding`` is the thin
ctypes layer with the same entry-point names. Importing the package does not load the library; the first
call does, and fails loudly if it has not been built (there is no CPU or PyTorch fallback).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
