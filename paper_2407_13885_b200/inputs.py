"""Seeded synthetic inputs and the five workload configurations.

This module holds NO attention or Softmax arithmetic: it only draws numbers.  It is the one
piece the CUDA path's harness and the CPU oracle's tests both use, and they meet only through
the arrays it returns (bfloat16 bit patterns as ``uint16`` for Q and K, ``float32`` for
precomputed scores).

Generator: counter-based, so any slice can be produced independently and reproducibly.
Counter ``c`` (one per pair of outputs) -> two SplitMix64 words -> two uniforms with 53 bits ->
Box-Muller -> times sigma -> float32 -> (for Q, K) round-to-nearest-even to bfloat16.

The paper measures on square random matrices with ``d_k = 128`` and states no value
distribution (Section VI-A, Section VII, Table I); these i.i.d. normal configurations stand
in for those workloads.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

SEED = 240713885
_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK = (1 << 64) - 1


def _mix(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on a uint64 array (wrap-around arithmetic)."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= _M1
    x ^= x >> np.uint64(27)
    x *= _M2
    x ^= x >> np.uint64(31)
    return x


def _stream_base(seed: int, stream_id: int) -> np.uint64:
    b = (seed * 0x9E3779B97F4A7C15 + (stream_id + 1) * 0xD1B54A32D192ED03) & _MASK
    return _mix(np.array([b], dtype=np.uint64))[0]


def normal_f32(seed: int, stream_id: int, count: int, sigma: float, offset: int = 0) -> np.ndarray:
    """``count`` float32 draws from N(0, sigma^2): elements ``offset .. offset+count`` of the
    stream ``(seed, stream_id)``.  Element ``e`` depends only on ``(seed, stream_id, e)``."""
    if count < 0 or offset < 0:
        raise ValueError("count and offset must be non-negative")
    out = np.empty(count, dtype=np.float32)
    if count == 0:
        return out
    base = _stream_base(seed, stream_id)
    first_pair = offset // 2
    last_pair = (offset + count + 1) // 2  # exclusive
    chunk = 1 << 22
    with np.errstate(over="ignore"):
        for p0 in range(first_pair, last_pair, chunk):
            p1 = min(p0 + chunk, last_pair)
            c = np.arange(p0, p1, dtype=np.uint64)
            w1 = _mix(base + (np.uint64(2) * c + np.uint64(1)) * _GAMMA)
            w2 = _mix(base + (np.uint64(2) * c + np.uint64(2)) * _GAMMA)
            u1 = ((w1 >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
            u2 = (w2 >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
            r = np.sqrt(-2.0 * np.log(u1))
            ang = (2.0 * math.pi) * u2
            pair = np.empty((p1 - p0, 2), dtype=np.float64)
            pair[:, 0] = r * np.cos(ang)
            pair[:, 1] = r * np.sin(ang)
            flat = (pair.reshape(-1) * float(sigma)).astype(np.float32)
            lo = max(offset, 2 * p0)
            hi = min(offset + count, 2 * p1)
            out[lo - offset:hi - offset] = flat[lo - 2 * p0:hi - 2 * p0]
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns.
    Inputs must be finite."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16_bits(seed: int, stream_id: int, count: int, sigma: float, offset: int = 0) -> np.ndarray:
    return f32_to_bf16_bits(normal_f32(seed, stream_id, count, sigma, offset))


@dataclass(frozen=True)
class Workload:
    """One benchmark/parity configuration."""
    name: str
    kind: str            # "fused" | "rows"
    B: int = 1
    H: int = 1
    N: int = 0           # sequence length (fused)
    d: int = 0           # head dimension (fused)
    rows: int = 0        # (rows)
    cols: int = 0        # (rows)
    sigma: float = 1.0
    scale: float = 1.0   # the float32 value handed to the kernel
    p_dtype: str = "bf16"  # "bf16" | "f32"
    cfg_id: int = 0

    @property
    def elements(self) -> int:
        if self.kind == "fused":
            return self.B * self.H * self.N * self.N
        return self.rows * self.cols

    @property
    def p_bytes(self) -> int:
        return self.elements * (2 if self.p_dtype == "bf16" else 4)

    @property
    def in_bytes(self) -> int:
        if self.kind == "fused":
            return 2 * self.B * self.H * self.N * self.d * 2
        return self.rows * self.cols * 4

    @property
    def flops(self) -> int:
        return 2 * self.elements * self.d if self.kind == "fused" else 0


def _f32(x: float) -> float:
    return float(np.float32(x))


WORKLOADS = {
    "c1": Workload("c1", "fused", B=1, H=1, N=256, d=64, sigma=1.0, scale=0.125, p_dtype="f32", cfg_id=1),
    "c2": Workload("c2", "fused", B=1, H=12, N=2048, d=64, sigma=1.0, scale=0.125, p_dtype="bf16", cfg_id=2),
    "c3": Workload("c3", "fused", B=4, H=32, N=4096, d=128, sigma=1.0,
                   scale=_f32(1.0 / math.sqrt(128.0)), p_dtype="bf16", cfg_id=3),
    "c4": Workload("c4", "rows", rows=8 * 4096, cols=8192, sigma=3.0, p_dtype="bf16", cfg_id=4),
    "c5": Workload("c5", "fused", B=1, H=8, N=16384, d=128, sigma=4.0,
                   scale=_f32(1.0 / math.sqrt(128.0)), p_dtype="bf16", cfg_id=5),
}


def make_qk(w: Workload, bh_begin: int = 0, bh_end: int | None = None, seed: int = SEED):
    """Q and K bit patterns for heads ``bh_begin .. bh_end`` (flattened b*H + h) of a fused
    workload, shaped ``[bh_end - bh_begin, N, d]``.  A slice equals the same slice of the whole."""
    if w.kind != "fused":
        raise ValueError("not a fused workload")
    bh_end = w.B * w.H if bh_end is None else bh_end
    per_head = w.N * w.d
    n = (bh_end - bh_begin) * per_head
    q = normal_bf16_bits(seed, 2 * w.cfg_id, n, w.sigma, offset=bh_begin * per_head)
    k = normal_bf16_bits(seed, 2 * w.cfg_id + 1, n, w.sigma, offset=bh_begin * per_head)
    shape = (bh_end - bh_begin, w.N, w.d)
    return q.reshape(shape), k.reshape(shape)


def make_scores(w: Workload, row_begin: int = 0, row_end: int | None = None, seed: int = SEED) -> np.ndarray:
    """float32 scores for rows ``row_begin .. row_end`` of a row-Softmax workload."""
    if w.kind != "rows":
        raise ValueError("not a row-Softmax workload")
    row_end = w.rows if row_end is None else row_end
    n = (row_end - row_begin) * w.cols
    s = normal_f32(seed, 2 * w.cfg_id, n, w.sigma, offset=row_begin * w.cols)
    return s.reshape(row_end - row_begin, w.cols)


def shard_range(total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous slice ``[begin, end)`` of ``total`` independent units owned by ``rank``:
    the quotient everywhere plus one extra unit on the first ``total % world`` ranks
    (the division-with-remainder rule of Section VI-B for rows over cores)."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard arguments")
    q, r = divmod(total, world)
    begin = rank * q + min(rank, r)
    return begin, begin + q + (1 if rank < r else 0)


def rank_heads(w: Workload, rank: int, world: int, scaling: str = "weak") -> tuple[int, int, int]:
    """Heads ``[begin, end)`` (flattened b*H + h) a rank computes, and the seed it draws them with.

    ``weak``: every rank owns a whole replica of the workload, drawn with its own seed (per-GPU work fixed).
    ``strong``: ONE workload; its heads are dealt out with :func:`shard_range` (quotient plus one extra head on the
    first ranks), every rank draws only its slice with the common seed, and no data crosses ranks: a head's rows
    need nothing from another head (Section VI-B's partition; Section VIII's "multiple cards")."""
    if scaling == "weak":
        return 0, w.B * w.H, SEED + rank
    if scaling == "strong":
        begin, end = shard_range(w.B * w.H, rank, world)
        return begin, end, SEED
    raise ValueError("scaling must be 'weak' or 'strong'")
