"""B200-native hierarchical, load-weighted gradient synchronisation (KAITIAN, Section III).

``paper_2505_10183_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/kaitian.h``); ``paper_2505_10183_b200.workloads`` holds the seeded synthetic
inputs.  The binding is imported on first use, and raises if the CUDA library has not
been built: there is no CPU fallback.
"""
from __future__ import annotations

import importlib

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in ("binding", "workloads", "build"):
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
