"""CPU oracle for attention weights / row Softmax (fp64, plain C, threaded over rows).

TEST INFRASTRUCTURE: importable only from ``tests/``, ``__graft_entry__.smoke()`` and
``bench.py``'s CPU-baseline / reference legs.  Nothing under ``paper_2407_13885_b200``
imports this package and this package imports nothing from there.

Each function is the definition written out in double precision:

* :func:`softmax_rows` - Softmax definition of Section VI with the max subtraction of Eq. 1.
* :func:`attnw` / :func:`attnw_rows` - ``softmax(scale * Q K^T)`` of Section IV (restated for
  ``n x d_k`` inputs and an ``n x n`` output in Section VII).
* :func:`project` - the linear transformation of the inputs into queries or keys (Section IV), ``X W_h`` per head.
* :func:`paper_cpu_softmax` - the fp32 single-core CPU program of Section VI-A (caching and
  recomputing forms), a timed context baseline, not the parity oracle.

Parity pins live in ``tests/test_oracle_pins.py``; none of them re-types the formula above:
they use invariants, closed forms, brute force in long double and float64 library routines.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_SOURCES = [os.path.join(_HERE, "oracle.c"), os.path.join(_HERE, "paper_cpu_softmax.c")]
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc into ``oracle/liboracle.so`` (no -ffast-math: IEEE order)."""
    newest = max(os.path.getmtime(s) for s in _SOURCES)
    if not force and os.path.exists(_LIB_PATH) and os.path.getmtime(_LIB_PATH) >= newest:
        return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", "-ffp-contract=off",
           "-o", tmp, *_SOURCES, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            c_long, c_int, c_float, vp = ctypes.c_long, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
            lib.oracle_softmax_rows.argtypes = [vp, vp, c_long, c_long, c_int]
            lib.oracle_softmax_rows_subset.argtypes = [vp, vp, c_long, vp, c_long, c_int]
            lib.oracle_attnw.argtypes = [vp, vp, vp, c_long, c_long, c_long, c_long, c_float, c_int]
            lib.oracle_attnw_rows.argtypes = [vp, vp, vp, c_long, c_long, c_long, c_long, c_float,
                                              vp, c_long, c_int]
            lib.oracle_scores_rows.argtypes = [vp, vp, vp, c_long, c_long, c_long, c_long, vp, c_long]
            lib.oracle_attn.argtypes = [vp, vp, vp, vp, c_long, c_long, c_long, c_long, c_float, c_int]
            lib.oracle_attn_rows.argtypes = [vp, vp, vp, vp, c_long, c_long, c_long, c_long, c_float,
                                             vp, c_long, c_int]
            lib.oracle_project.argtypes = [vp, vp, vp, c_long, c_long, c_long, c_long, c_long, vp, c_long]
            lib.oracle_project.restype = c_int
            for f in (lib.oracle_softmax_rows, lib.oracle_softmax_rows_subset, lib.oracle_attnw,
                      lib.oracle_attnw_rows, lib.oracle_scores_rows, lib.oracle_attn, lib.oracle_attn_rows):
                f.restype = c_int
            lib.paper_cpu_softmax_caching_f32.argtypes = [vp, vp, c_long, c_long]
            lib.paper_cpu_softmax_recomputing_f32.argtypes = [vp, vp, c_long, c_long]
            lib.paper_cpu_softmax_caching_f32.restype = None
            lib.paper_cpu_softmax_recomputing_f32.restype = None
            _lib = lib
    return _lib


def host_cores() -> int:
    """Cores this process may run on (what the threaded oracle uses by default)."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def _as_bf16_bits(x, name: str) -> np.ndarray:
    a = np.ascontiguousarray(x)
    if a.dtype != np.uint16:
        raise TypeError(f"{name} must hold bfloat16 bit patterns as uint16, got {a.dtype}")
    return a


def softmax_rows(S, rows_subset=None, threads: int | None = None) -> np.ndarray:
    """Row Softmax (Section VI, Eq. 1) of float32 scores ``S[rows, cols]`` -> float64.

    ``rows_subset``: optional 1-D array of row indices; only those rows are computed."""
    S = np.ascontiguousarray(S)
    if S.dtype != np.float32 or S.ndim != 2:
        raise TypeError("S must be a 2-D float32 array")
    threads = threads or host_cores()
    rows, cols = S.shape
    lib = _load()
    if rows_subset is None:
        P = np.empty((rows, cols), dtype=np.float64)
        _check(lib.oracle_softmax_rows(_ptr(S), _ptr(P), rows, cols, threads), "softmax_rows")
        return P
    ids = np.ascontiguousarray(rows_subset, dtype=np.int64)
    if ids.size and (ids.min() < 0 or ids.max() >= rows):
        raise IndexError("row index out of range")
    P = np.empty((ids.size, cols), dtype=np.float64)
    _check(lib.oracle_softmax_rows_subset(_ptr(S), _ptr(P), cols, _ptr(ids), ids.size, threads),
           "softmax_rows_subset")
    return P


def attnw(Q, K, scale: float, threads: int | None = None) -> np.ndarray:
    """``softmax(scale * Q K^T)`` (Section IV) for bf16 bit patterns ``Q, K [B,H,N,d]`` -> float64
    ``[B,H,N,N]``."""
    Q = _as_bf16_bits(Q, "Q")
    K = _as_bf16_bits(K, "K")
    if Q.shape != K.shape or Q.ndim != 4:
        raise ValueError("Q and K must both be [B,H,N,d]")
    B, H, N, d = Q.shape
    P = np.empty((B, H, N, N), dtype=np.float64)
    _check(_load().oracle_attnw(_ptr(Q), _ptr(K), _ptr(P), B, H, N, d, float(np.float32(scale)),
                                threads or host_cores()), "attnw")
    return P


def attnw_rows(Q, K, scale: float, row_ids, threads: int | None = None) -> np.ndarray:
    """Selected rows of :func:`attnw`.  ``row_ids`` are global row numbers ``(b*H + h)*N + i``;
    returns float64 ``[len(row_ids), N]``."""
    Q = _as_bf16_bits(Q, "Q")
    K = _as_bf16_bits(K, "K")
    if Q.shape != K.shape or Q.ndim != 4:
        raise ValueError("Q and K must both be [B,H,N,d]")
    B, H, N, d = Q.shape
    ids = np.ascontiguousarray(row_ids, dtype=np.int64)
    P = np.empty((ids.size, N), dtype=np.float64)
    _check(_load().oracle_attnw_rows(_ptr(Q), _ptr(K), _ptr(P), B, H, N, d,
                                     float(np.float32(scale)), _ptr(ids), ids.size,
                                     threads or host_cores()), "attnw_rows")
    return P


def attn(Q, K, V, scale: float, row_ids=None, threads: int | None = None) -> np.ndarray:
    """``softmax(scale * Q K^T) V`` (Section IV) for bf16 bit patterns ``Q, K, V [B,H,N,d]`` -> float64
    ``[B,H,N,d]``, or ``[len(row_ids), d]`` for the listed global rows ``(b*H + h)*N + i``."""
    Q = _as_bf16_bits(Q, "Q")
    K = _as_bf16_bits(K, "K")
    V = _as_bf16_bits(V, "V")
    if Q.shape != K.shape or Q.shape != V.shape or Q.ndim != 4:
        raise ValueError("Q, K and V must all be [B,H,N,d]")
    B, H, N, d = Q.shape
    if row_ids is None:
        O = np.empty((B, H, N, d), dtype=np.float64)
        _check(_load().oracle_attn(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), B, H, N, d, float(np.float32(scale)),
                                   threads or host_cores()), "attn")
        return O
    ids = np.ascontiguousarray(row_ids, dtype=np.int64)
    O = np.empty((ids.size, d), dtype=np.float64)
    _check(_load().oracle_attn_rows(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), B, H, N, d, float(np.float32(scale)),
                                    _ptr(ids), ids.size, threads or host_cores()), "attn_rows")
    return O


def project(X, W, row_ids=None) -> np.ndarray:
    """Queries (or keys) from the inputs (Section IV): ``out[b,h,n,c] = sum_m X[b,n,m] W[h,c,m]`` for bf16 bit
    patterns ``X [B,N,d_model]`` and ``W [H,d,d_model]`` (row ``c`` of head ``h`` is column ``c`` of that head's
    parameter matrix) -> float64 ``[B,H,N,d]``, or ``[len(row_ids), d]`` for the listed global rows
    ``(b*H + h)*N + n``."""
    X = _as_bf16_bits(X, "X")
    W = _as_bf16_bits(W, "W")
    if X.ndim != 3 or W.ndim != 3 or X.shape[2] != W.shape[2]:
        raise ValueError("X must be [B,N,d_model] and W [H,d,d_model]")
    B, N, d_model = X.shape
    H, d, _ = W.shape
    if row_ids is None:
        out = np.empty((B, H, N, d), dtype=np.float64)
        _check(_load().oracle_project(_ptr(X), _ptr(W), _ptr(out), B, N, d_model, H, d, None, 0), "project")
        return out
    ids = np.ascontiguousarray(row_ids, dtype=np.int64)
    out = np.empty((ids.size, d), dtype=np.float64)
    _check(_load().oracle_project(_ptr(X), _ptr(W), _ptr(out), B, N, d_model, H, d, _ptr(ids), ids.size), "project")
    return out


def scores_rows(Q, K, row_ids) -> np.ndarray:
    """Unscaled scores ``sum_c Q_ic K_jc`` of selected global rows -> float64 ``[len, N]``."""
    Q = _as_bf16_bits(Q, "Q")
    K = _as_bf16_bits(K, "K")
    B, H, N, d = Q.shape
    ids = np.ascontiguousarray(row_ids, dtype=np.int64)
    S = np.empty((ids.size, N), dtype=np.float64)
    _check(_load().oracle_scores_rows(_ptr(Q), _ptr(K), _ptr(S), B, H, N, d, _ptr(ids), ids.size),
           "scores_rows")
    return S


def paper_cpu_softmax(Z, variant: str = "caching") -> np.ndarray:
    """Section VI-A's CPU program (fp32, one core).  ``variant``: "caching" | "recomputing"."""
    Z = np.ascontiguousarray(Z)
    if Z.dtype != np.float32 or Z.ndim != 2:
        raise TypeError("Z must be a 2-D float32 array")
    out = np.empty_like(Z)
    lib = _load()
    fn = {"caching": lib.paper_cpu_softmax_caching_f32,
          "recomputing": lib.paper_cpu_softmax_recomputing_f32}[variant]
    fn(_ptr(Z), _ptr(out), Z.shape[0], Z.shape[1])
    return out
