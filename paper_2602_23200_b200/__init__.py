"""InnerQ decode attention for B200 (sm_100a): ctypes binding over the C-ABI CUDA library.

`synth` (seeded inputs) is importable on its own; the CUDA binding is loaded lazily on
first attribute access so that host-only tools can import this package without a GPU.
"""
from importlib import import_module

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name in ("binding", "synth"):
        return import_module(f"{__name__}.{name}")
    raise AttributeError(name)
