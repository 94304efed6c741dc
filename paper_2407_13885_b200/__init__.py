"""Attention weights ``P = Softmax(scale * Q K^T)`` on B200 (sm_100a).

Two operations, both hand-written CUDA behind a C-ABI shared library (``include/attnw.h``):

* ``attnw_fused`` - matmul, scaling and Softmax in one kernel (the fused kernel of
  Section VII of the paper, re-designed for tcgen05 / TMEM / TMA);
* ``softmax_rows`` - the dedicated row-Softmax kernel over precomputed scores
  (Section VI-B).

The Python layer only marshals pointers; there is no CPU or PyTorch fallback - calling an
operation without the compiled library raises.
"""
from __future__ import annotations

__all__ = ["attnw_fused", "softmax_rows", "binding", "inputs", "build"]


def __getattr__(name):  # lazy: importing the package never needs the compiled library
    if name in ("attnw_fused", "softmax_rows", "AttnwError", "query_status", "strerror",
                "version", "library_path", "host_attnw_fused", "host_softmax_rows"):
        from . import binding
        return getattr(binding, name)
    if name in ("binding", "inputs", "build"):
        import importlib
        return importlib.import_module(f".{name}", __name__)
    raise AttributeError(name)
