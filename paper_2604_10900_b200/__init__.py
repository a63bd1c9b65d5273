"""B200-native compression event of CASK (core-aware selective KV compression).

``workloads`` (numpy only) generates the seeded synthetic caches; ``binding``
is the thin ctypes layer over the C-ABI library ``libcask.so`` built from
``csrc/``.  The binding is loaded on first use and raises if the CUDA library
is missing: there is no CPU fallback.
"""
from __future__ import annotations

import importlib

__all__ = ["workloads", "binding", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
