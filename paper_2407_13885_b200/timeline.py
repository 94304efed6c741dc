"""Per-phase cycle table of the grid-row kernel (the analogue of the paper's per-operation runtime figures, Fig. 4 / 5).

Builds an instrumented copy of the library beside the product one (``-DATTNW_TIMELINE=<CTA>``: one lane per role of
that CTA stamps ``clock64()`` per row block), runs a reduced case of the headline shape through it and prints where
the cycles of a row block go.  The product library carries none of the instrumentation.

    python -m paper_2407_13885_b200.timeline [--cta 1] [--heads 64] [--n 4096] [--d 128]

or ``python bench.py --timeline``.  Prints one JSON line (``"timeline_run": true``); never a benchmark value.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os

import numpy as np

from . import build as _build

TIMELINE_LIB = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libattnw_timeline.so")
EVENTS, SLOTS = 32, 160


def _load(cta: int) -> ctypes.CDLL:
    _build.build_library(force=True, defines=(f"ATTNW_TIMELINE={cta}",), out=TIMELINE_LIB)
    lib = ctypes.CDLL(TIMELINE_LIB)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.attnw_fused.argtypes = [vp, vp, vp, ci, ci, ci, ci, ctypes.c_float, vp]
    lib.attnw_fused.restype = ci
    lib.attnw_set_fused_variant.argtypes = [ci]
    lib.attnw_query_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint)]
    lib.attnw_debug_timeline.argtypes = [vp]
    return lib


def run(cta: int = 1, heads: int = 64, n: int = 4096, d: int = 128, launches: int = 10) -> dict:
    import torch
    lib = _load(cta)
    q = torch.randn(1, heads, n, d, device="cuda").to(torch.bfloat16)
    k = torch.randn(1, heads, n, d, device="cuda").to(torch.bfloat16)
    p = torch.empty((1, heads, n, n), dtype=torch.bfloat16, device="cuda")
    if lib.attnw_set_fused_variant(4) != 0:
        raise RuntimeError("attnw_set_fused_variant(4) failed")
    scale = 1.0 / math.sqrt(d)
    for _ in range(launches):
        rc = lib.attnw_fused(q.data_ptr(), k.data_ptr(), p.data_ptr(), 1, heads, n, d, scale, None)
        if rc != 0:
            raise RuntimeError(f"attnw_fused: status {rc}")
    torch.cuda.synchronize()
    word = ctypes.c_uint(0)
    if lib.attnw_query_status(None, ctypes.byref(word)) != 0:
        raise RuntimeError(f"device status word {word.value:#x}")
    buf = np.zeros((EVENTS, SLOTS), dtype=np.int64)
    if lib.attnw_debug_timeline(buf.ctypes.data) != 0:
        raise RuntimeError("attnw_debug_timeline failed")
    group_ctas = (n + 255) // 256
    groups = max(1, min(torch.cuda.get_device_properties(0).multi_processor_count // group_ctas, heads * ((n + 127) // 128)))
    items = heads * ((n + 127) // 128) // groups
    lo, hi = 8, min(items - 2, SLOTS - 2)
    if hi - lo < 4:
        raise RuntimeError("too few row blocks per group for a steady-state window; raise --heads")
    it = np.arange(lo, hi)

    def span(a, b):  # mean cycles from event a to event b of the same row block
        return float(np.mean(buf[b, it] - buf[a, it]))

    period = float(np.mean(np.diff(buf[13, lo:hi])))
    table = {
        "period_per_row_block": period,
        "exponential_role": {
            "slot0_ready_to_halves_posted": span(2, 4),
            "box0_load_and_maximum": span(17, 16), "box0_exponentials": span(16, 18), "box0_wait_region_and_store": span(18, 24),
            "box1_load_and_maximum": span(20, 19), "box1_exponentials": span(19, 21), "box1_wait_region_and_store": span(21, 26),
            "mma_issue_to_exponentials_begin": span(13, 0),
        },
        "normalise_role": {
            "first_warp_done_to_block_visible_to_normalise": float(np.mean(buf[6, it] - buf[4, it])),
            "wait_for_group": span(6, 11), "reduce_and_read_box0": span(11, 12),
            "box2_wait_staging": span(14, 15), "box2_scale_round_stage": span(15, 8), "box2_fence_and_hand_over": span(8, 9),
            "all_pairs_seen_to_block_done": span(11, 7),
        },
    }
    return {"timeline_run": True, "case": f"attnw_fused (grid-row kernel) B=1 H={heads} N={n} d={d}, CTA {cta}, "
                                          f"row blocks {lo}..{hi - 1} of {items} in its group's list",
            "unit": "SM cycles (clock64), means over the window", "cycles": table}


def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--cta", type=int, default=1)
    ap.add_argument("--heads", type=int, default=64)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--d", type=int, default=128, choices=[64, 128])
    a = ap.parse_args(argv)
    print(json.dumps(run(a.cta, a.heads, a.n, a.d)))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
