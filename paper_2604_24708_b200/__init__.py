"""HDET hot path for one B200: a C-ABI CUDA library (csrc/, include/hdet.h) and its ctypes binding.

``from paper_2604_24708_b200 import binding`` loads ``lib/libhdet.so`` and fails if it has not
been built (``python -m paper_2604_24708_b200.build``); there is no CPU fallback.
"""
import importlib

__all__ = ["binding", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
