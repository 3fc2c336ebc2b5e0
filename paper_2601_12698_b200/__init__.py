"""Template-plus-search tuner for the fused residual-add + RMSNorm kernel on sm_100a.

``synth`` (seeded inputs) imports on any machine.  ``binding`` loads the CUDA
shared library and is imported lazily, so that input generation does not
require the library to be built.
"""
from __future__ import annotations

import importlib

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
