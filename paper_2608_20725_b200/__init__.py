"""B200-native im2win convolution: im2win transform + fp32 / fp16 forward convolution.

The compute path lives in ``csrc/`` (CUDA for sm_100a behind a C ABI declared
in ``include/im2win.h``); ``binding`` marshals torch tensors into that ABI.
Importing the package does not load the library; the first call does, and it
raises if the library cannot be built or loaded (there is no CPU fallback).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        import importlib
        return importlib.import_module(f".{name}", __name__)
    raise AttributeError(name)
