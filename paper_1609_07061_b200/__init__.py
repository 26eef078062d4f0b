"""B200-native forward hot path of quantised / binarised neural networks.

The product is the C-ABI library ``libqnn.so`` (hand-written sm_100a CUDA
kernels, declared in ``include/qnn.h``); ``binding`` is a thin ctypes layer with
the same names that only marshals arguments.  ``workloads`` draws seeded
synthetic inputs and contains none of the method's arithmetic.

The binding is loaded on first use of any ``qnn_*`` name and raises if the
library has not been built: there is no CPU fallback.
"""
from __future__ import annotations

import importlib

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in ("binding", "workloads", "build"):
        return importlib.import_module(f"{__name__}.{name}")
    if name.startswith("qnn_") or name.startswith("QNN_"):
        return getattr(importlib.import_module(f"{__name__}.binding"), name)
    raise AttributeError(name)
