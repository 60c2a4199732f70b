"""B200-native cold-start convolution path (NNV12's hot path) -- Python side.

`binding` mirrors the C ABI of libnnv.so one to one; `harness` is a thin
PyTorch helper that owns device memory, pinned host blobs and streams.  The
library must be built first (`python -m paper_2206_07446_b200.build`); there is
no fallback when it is missing.
"""
import importlib

__all__ = ["binding", "harness", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
