"""ctypes binding of ``libattnw.so`` - argument marshalling only.

Every operation runs in the library's CUDA kernels; nothing here computes.  If the compiled
library is missing the import of this module raises: there is no fallback.  PyTorch is used
for device memory and streams only (``tensor.data_ptr()``, ``torch.cuda.current_stream()``).
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

_vp, _int, _ll, _float = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_float

# name -> (restype, argtypes); mirrors include/attnw.h one to one
SIGNATURES = {
    "attn_fused": (_int, [_vp, _vp, _vp, _vp, _int, _int, _int, _int, _float, _vp]),
    "attnw_project_qk": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _int, _int, _int, _int, _vp]),
    "attnw_fused": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, _float, _vp]),
    "attnw_fused_f32": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, _float, _vp]),
    "softmax_rows": (_int, [_vp, _vp, _ll, _ll, _vp]),
    "softmax_rows_f32": (_int, [_vp, _vp, _ll, _ll, _vp]),
    "attnw_fused_host": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, _float, _int]),
    "softmax_rows_host": (_int, [_vp, _vp, _ll, _ll, _int]),
    "attnw_host_release": (_int, []),
    "attnw_fused_noalloc": (_int, [_vp, _vp, _vp, _int, _int, _int, _int, ctypes.c_float, _vp]),
    "attnw_query_status": (_int, [_vp, ctypes.POINTER(ctypes.c_uint)]),
    "attnw_selftest_wait_timeout": (_int, [_ll, _vp]),
    "attnw_set_fused_variant": (_int, [_int]),
    "attnw_set_attn_variant": (_int, [_int]),
    "attnw_set_rows_variant": (_int, [_int]),
    "attnw_launch_count": (_ll, [_int]),
    "attnw_strerror": (ctypes.c_char_p, [_int]),
    "attnw_version": (_int, []),
}


def library_path() -> str:
    return _build.LIB_PATH


def _load() -> ctypes.CDLL:
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2407_13885_b200.build` "
            "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(path)
    for name, (restype, argtypes) in SIGNATURES.items():
        fn = getattr(lib, name)  # AttributeError if the library lacks a declared symbol
        fn.restype = restype
        fn.argtypes = argtypes
    return lib


lib = _load()


class AttnwError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: attnw status {code}: {strerror(code)}")


def strerror(code: int) -> str:
    return lib.attnw_strerror(int(code)).decode()


def version() -> int:
    return int(lib.attnw_version())


FUSED_VARIANTS = {"auto": 0, "two_pass": 1, "resident": 2, "resident_owner": 3, "gridrow": 4}


def set_fused_variant(variant: str | int) -> None:
    """Selects the kernel behind ``attnw_fused``: "auto" (by shape), "two_pass", "resident", "resident_owner"
    (the resident kernel with the reduce-and-broadcast exchange) or "gridrow" (groups of CTAs of a cooperative grid)."""
    code = FUSED_VARIANTS[variant] if isinstance(variant, str) else int(variant)
    _check(lib.attnw_set_fused_variant(code), "attnw_set_fused_variant")


ROWS_VARIANTS = {"auto": 0, "caching": 1, "recomputing": 2, "recomputing_registers": 3}


def set_rows_variant(variant: str | int) -> None:
    """Selects the form of ``softmax_rows``: "auto" (by row length), "caching", "recomputing" (second read) or
    "recomputing_registers" (Section VI-A)."""
    code = ROWS_VARIANTS[variant] if isinstance(variant, str) else int(variant)
    _check(lib.attnw_set_rows_variant(code), "attnw_set_rows_variant")


ATTN_VARIANTS = {"auto": 0, "two_pass": 1, "one_pass": 2}


def set_attn_variant(variant: str | int) -> None:
    """Selects the kernel behind ``attn_fused``: "auto" (the one-pass kernel), "two_pass" or "one_pass"."""
    code = ATTN_VARIANTS[variant] if isinstance(variant, str) else int(variant)
    _check(lib.attnw_set_attn_variant(code), "attnw_set_attn_variant")


def launch_count(reset: bool = False) -> int:
    return int(lib.attnw_launch_count(1 if reset else 0))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _check(code: int, where: str) -> None:
    if code != 0:
        raise AttnwError(code, where)


def _require_cuda(t: torch.Tensor, name: str, dtype) -> None:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


def attnw_fused(Q: torch.Tensor, K: torch.Tensor, scale: float, P: torch.Tensor | None = None,
                out_dtype: torch.dtype = torch.bfloat16, stream=None) -> torch.Tensor:
    """``P = Softmax(scale * Q K^T)`` over the last axis, one fused kernel.

    ``Q, K``: CUDA bfloat16 ``[B, H, N, d]``; returns ``P [B, H, N, N]`` (bfloat16 or float32).
    Asynchronous on ``stream`` (default: torch's current stream)."""
    _require_cuda(Q, "Q", torch.bfloat16)
    _require_cuda(K, "K", torch.bfloat16)
    if Q.dim() != 4 or Q.shape != K.shape:
        raise ValueError("Q and K must both be [B, H, N, d]")
    B, H, N, d = Q.shape
    if P is None:
        P = torch.empty((B, H, N, N), dtype=out_dtype, device=Q.device)
    else:
        _require_cuda(P, "P", P.dtype)
        if tuple(P.shape) != (B, H, N, N) or P.dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("P must be [B, H, N, N] in bfloat16 or float32")
    fn = lib.attnw_fused if P.dtype == torch.bfloat16 else lib.attnw_fused_f32
    with torch.cuda.device(Q.device):
        _check(fn(Q.data_ptr(), K.data_ptr(), P.data_ptr(), B, H, N, d, float(scale), _stream_ptr(stream)),
               "attnw_fused")
    return P


def attn_fused(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, scale: float, O: torch.Tensor | None = None,
               stream=None) -> torch.Tensor:
    """``O = Softmax(scale * Q K^T) V`` in one fused kernel; ``Q, K, V, O``: CUDA bfloat16 ``[B, H, N, d]``.
    Asynchronous on ``stream`` (default: torch's current stream)."""
    for t, name in ((Q, "Q"), (K, "K"), (V, "V")):
        _require_cuda(t, name, torch.bfloat16)
    if Q.dim() != 4 or Q.shape != K.shape or Q.shape != V.shape:
        raise ValueError("Q, K and V must all be [B, H, N, d]")
    B, H, N, d = Q.shape
    if O is None:
        O = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=Q.device)
    else:
        _require_cuda(O, "O", torch.bfloat16)
        if tuple(O.shape) != (B, H, N, d):
            raise ValueError("O must be [B, H, N, d]")
    with torch.cuda.device(Q.device):
        _check(lib.attn_fused(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), B, H, N, d, float(scale),
                              _stream_ptr(stream)), "attn_fused")
    return O


def project_qk(X: torch.Tensor, Wq: torch.Tensor, Wk: torch.Tensor, Q: torch.Tensor | None = None,
               K: torch.Tensor | None = None, stream=None) -> tuple[torch.Tensor, torch.Tensor]:
    """Queries and keys from the inputs: ``Q[b,h] = X[b] Wq[h]^T``, ``K[b,h] = X[b] Wk[h]^T`` for CUDA bfloat16
    ``X [B, N, d_model]`` and ``Wq, Wk [H, d, d_model]`` -> ``Q, K [B, H, N, d]`` (bfloat16), the layout
    ``attnw_fused`` and ``attn_fused`` read.  Asynchronous on ``stream`` (default: torch's current stream)."""
    for t, name in ((X, "X"), (Wq, "Wq"), (Wk, "Wk")):
        _require_cuda(t, name, torch.bfloat16)
    if X.dim() != 3 or Wq.dim() != 3 or Wq.shape != Wk.shape or Wq.shape[2] != X.shape[2]:
        raise ValueError("X must be [B, N, d_model] and Wq, Wk [H, d, d_model]")
    B, N, d_model = X.shape
    H, d, _ = Wq.shape
    outs = []
    for t, name in ((Q, "Q"), (K, "K")):
        if t is None:
            t = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=X.device)
        else:
            _require_cuda(t, name, torch.bfloat16)
            if tuple(t.shape) != (B, H, N, d):
                raise ValueError(f"{name} must be [B, H, N, d]")
        outs.append(t)
    with torch.cuda.device(X.device):
        _check(lib.attnw_project_qk(X.data_ptr(), Wq.data_ptr(), Wk.data_ptr(), outs[0].data_ptr(), outs[1].data_ptr(), B, N,
                                    d_model, H, d, _stream_ptr(stream)), "attnw_project_qk")
    return outs[0], outs[1]


def softmax_rows(S: torch.Tensor, P: torch.Tensor | None = None, out_dtype: torch.dtype = torch.bfloat16,
                 stream=None) -> torch.Tensor:
    """Row-wise Softmax of float32 scores ``S [rows, cols]`` -> ``P`` (bfloat16 or float32)."""
    _require_cuda(S, "S", torch.float32)
    if S.dim() != 2:
        raise ValueError("S must be [rows, cols]")
    rows, cols = S.shape
    if P is None:
        P = torch.empty((rows, cols), dtype=out_dtype, device=S.device)
    else:
        _require_cuda(P, "P", P.dtype)
        if tuple(P.shape) != (rows, cols) or P.dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("P must be [rows, cols] in bfloat16 or float32")
    fn = lib.softmax_rows if P.dtype == torch.bfloat16 else lib.softmax_rows_f32
    with torch.cuda.device(S.device):
        _check(fn(S.data_ptr(), P.data_ptr(), rows, cols, _stream_ptr(stream)), "softmax_rows")
    return P


def _require_host(t: torch.Tensor, name: str, dtype) -> None:
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a CPU tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous with dtype {dtype}")


def host_attnw_fused(Q: torch.Tensor, K: torch.Tensor, scale: float, P: torch.Tensor) -> torch.Tensor:
    """Host-memory variant: copies in, computes, copies ``P`` back; returns when ``P`` is complete."""
    _require_host(Q, "Q", torch.bfloat16)
    _require_host(K, "K", torch.bfloat16)
    B, H, N, d = Q.shape
    if P.is_cuda or not P.is_contiguous() or tuple(P.shape) != (B, H, N, N):
        raise ValueError("P must be a contiguous CPU tensor [B, H, N, N]")
    f32 = {torch.bfloat16: 0, torch.float32: 1}[P.dtype]
    _check(lib.attnw_fused_host(Q.data_ptr(), K.data_ptr(), P.data_ptr(), B, H, N, d, float(scale), f32),
           "attnw_fused_host")
    return P


def host_softmax_rows(S: torch.Tensor, P: torch.Tensor) -> torch.Tensor:
    _require_host(S, "S", torch.float32)
    rows, cols = S.shape
    if P.is_cuda or not P.is_contiguous() or tuple(P.shape) != (rows, cols):
        raise ValueError("P must be a contiguous CPU tensor [rows, cols]")
    f32 = {torch.bfloat16: 0, torch.float32: 1}[P.dtype]
    _check(lib.softmax_rows_host(S.data_ptr(), P.data_ptr(), rows, cols, f32), "softmax_rows_host")
    return P


def host_release() -> None:
    _check(lib.attnw_host_release(), "attnw_host_release")


def query_status(stream=None) -> int:
    """Synchronises ``stream`` and returns the device status word (0 = healthy); clears it."""
    word = ctypes.c_uint(0)
    code = lib.attnw_query_status(_stream_ptr(stream), ctypes.byref(word))
    if code not in (0, 6):
        raise AttnwError(code, "attnw_query_status")
    return int(word.value)


def selftest_wait_timeout(limit_cycles: int = 1_000_000, stream=None) -> None:
    """Launches the failure-path self-test: one warp waits ``limit_cycles`` SM clocks on a barrier nobody arrives on,
    gives up and records site 127 in the device status word (see ``attnw_selftest_wait_timeout``)."""
    _check(lib.attnw_selftest_wait_timeout(int(limit_cycles), _stream_ptr(stream)), "attnw_selftest_wait_timeout")


def attnw_fused_noalloc(Q: torch.Tensor, K: torch.Tensor, scale: float, P: torch.Tensor | None = None,
                        stream=None) -> torch.Tensor:
    """``attnw_fused`` (bfloat16 P, N <= 4096) through the entry point that never allocates device memory: for callers
    that may not call cudaMalloc (a memory pool owns the device, or the call sits in a latency-critical loop).  The
    output tensor is still the caller's (or allocated here by torch, outside the library)."""
    _require_cuda(Q, "Q", torch.bfloat16)
    _require_cuda(K, "K", torch.bfloat16)
    if Q.dim() != 4 or Q.shape != K.shape:
        raise ValueError("Q and K must both be [B, H, N, d]")
    B, H, N, d = Q.shape
    if P is None:
        P = torch.empty((B, H, N, N), dtype=torch.bfloat16, device=Q.device)
    else:
        _require_cuda(P, "P", torch.bfloat16)
        if tuple(P.shape) != (B, H, N, N):
            raise ValueError("P must be [B, H, N, N] in bfloat16")
    with torch.cuda.device(Q.device):
        _check(lib.attnw_fused_noalloc(Q.data_ptr(), K.data_ptr(), P.data_ptr(), B, H, N, d, float(scale),
                                       _stream_ptr(stream)), "attnw_fused_noalloc")
    return P
