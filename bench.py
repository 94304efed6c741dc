#!/usr/bin/env python
"""Benchmark of the fused attention-weight kernel (and, beside it, the dedicated row-Softmax kernel).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one launch of ``attnw_fused`` over the whole headline workload (fused, B=4, H=32,
N=4096, d=128, bf16 -> bf16 P): matmul, scaling, statistics pass, normalise pass and the store of P.
``value`` is attention-weight elements per second with inputs resident in HBM; ``e2e`` is the same
metric through the host-buffer C-ABI call (host->device and device->host copies inside the timed
region).  With N > 1 (torchrun) every rank runs the full workload on its own seeded inputs (heads are
independent, no collective on the data path): weak scaling, time = max over ranks.

``--impl reference`` times the CPU oracle on the host cores on a bounded sample of the same workload.
Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "attention-weight elements/sec"
UNIT = "elements/s"
HEADLINE = "c3"
# Fallback peaks (an earlier measurement on this machine) used only when MEASURED_PEAKS.json is absent.
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
# Measured traffic per launch comes from profiles/ncu_traffic.json, which every capture summarised under profiles/
# updates (bytes per head or per row of the reduced case, scaled here by the units one full launch processes).
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")


def measured_traffic(kernel_key: str, units: float):
    """Bytes one launch moves according to the ncu capture of `kernel_key` (DRAM reads + bytes the SMs wrote towards
    L2: the DRAM write counter misses what is still dirty in L2 when the kernel ends), or None without a capture."""
    try:
        with open(TRAFFIC_FILE) as f:
            entry = json.load(f)[kernel_key]
        return float(entry["bytes_per_unit"]) * units
    except Exception:
        return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
                "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples: list[int] = []
        self.reason_bits = 0
        self.sm_max = None
        self.halt = threading.Event()
        self.handle = None
        self.nvml = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            handle = None
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.handle = handle
            self.nvml = pynvml
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def _reasons(self) -> int:
        n = self.nvml
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            fn = getattr(n, name, None)
            if fn is not None:
                try:
                    return int(fn(self.handle))
                except Exception:
                    continue
        return 0

    def run(self):
        if self.handle is None:
            return
        n = self.nvml
        while not self.halt.is_set():
            try:
                self.samples.append(int(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                self.reason_bits |= self._reasons()
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self) -> dict:
        if self.handle is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0,
                    "note": "NVML unavailable" if self.handle is None else "no samples"}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(self.samples)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
# ------------------------------------------------------------------------------------------

def oracle_sample_rate(w, target_seconds: float, seed_offset: int = 0):
    """Times the oracle, as it stands, on complete rows of the workload; returns (elements/s, info)."""
    import oracle
    from paper_2407_13885_b200 import inputs
    cores = oracle.host_cores()
    heads = min(2, w.B * w.H)
    q, k = inputs.make_qk(w, 0, heads)
    q = q.reshape(1, heads, w.N, w.d)
    k = k.reshape(1, heads, w.N, w.d)
    rng = np.random.default_rng(1234 + seed_offset)
    probe = max(cores * 8, 64)
    ids = rng.integers(0, heads * w.N, size=probe)
    t0 = time.perf_counter()
    oracle.attnw_rows(q, k, w.scale, ids)
    dt = time.perf_counter() - t0
    per_row = dt / probe
    n_rows = int(min(max(probe, target_seconds / max(per_row, 1e-9)), 1 << 22))
    ids = rng.integers(0, heads * w.N, size=n_rows)
    t0 = time.perf_counter()
    oracle.attnw_rows(q, k, w.scale, ids)
    dt = time.perf_counter() - t0
    value = n_rows * w.N / dt
    info = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_rows} complete rows (N={w.N}, d={w.d}) drawn from {heads} heads of {w.name}, "
                      f"{dt:.2f} s wall, fp64, threaded over rows"}
    return value, info, dt, n_rows


def paper_cpu_rows_line(target_seconds: float = 2.0):
    """The CPU program of Section VI-A as the paper ran it - C, 32-bit floats, ONE core, caching and recomputing forms
    - on rows of the row-Softmax configuration c4 (8192 columns), a bounded sample each: the neighbour of the two CPU
    columns of Table I on this host.  Context beside the oracle line, not a target."""
    import oracle
    from paper_2407_13885_b200 import inputs
    w = inputs.WORKLOADS["c4"]
    out = {"workload": f"c4 rows: float32 scores [rows x {w.cols}], N(0,{w.sigma:g}^2)", "cores": 1, "kind": "paper_cpu_program",
           "unit": UNIT}
    rows = 1024
    Z = inputs.make_scores(w, 0, rows)
    for form in ("caching", "recomputing"):
        reps, dt = 0, 0.0
        while dt < target_seconds and reps < 64:
            t0 = time.perf_counter()
            oracle.paper_cpu_softmax(Z, form)
            dt += time.perf_counter() - t0
            reps += 1
        out[form] = {"value": reps * rows * w.cols / dt, "rows": rows, "passes": reps, "seconds": dt}
    out["caching_over_recomputing"] = out["caching"]["value"] / out["recomputing"]["value"]
    return out


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    from paper_2407_13885_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    # seconds of CPU work per step, bounded so that the whole run ends within a few minutes
    per_step = max(0.2, min(4.0, 150.0 / max(args.steps + args.warmup, 1)))
    for i in range(args.warmup):
        oracle_sample_rate(w, 0.5, seed_offset=i)
    total_t, total_rows, info = 0.0, 0, None
    for i in range(args.steps):
        _, info, dt, n_rows = oracle_sample_rate(w, per_step, seed_offset=100 + i)
        total_t += dt
        total_rows += n_rows
    value = total_rows * w.N / total_t
    info["value"] = value
    info["sample"] = (f"each step = about {per_step:.0f} s of oracle work on complete rows of {w.name} "
                      f"({total_rows} rows over {args.steps} steps)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, 1),
            "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def workload_config(w, world, scaling="weak"):
    cfg = {"workload": f"{w.name}: fused attention weights B={w.B} H={w.H} N={w.N} d={w.d}, Q,K bf16 N(0,{w.sigma:g}^2), "
                       f"scale={w.scale:.9g}, P {w.p_dtype}",
           "B": w.B, "H": w.H, "N": w.N, "d": w.d, "p_dtype": w.p_dtype,
           "parallelism": (f"{world} x independent replicas of the workload (heads are independent; no collective)"
                           if scaling == "weak" else
                           f"the workload's {w.B * w.H} heads dealt out over {world} ranks (quotient + remainder on the first "
                           "ranks; heads are independent; no collective)"),
           "l2": "no flush: each launch streams 4.56 GB (Q+K 268 MB, P 4.29 GB), far beyond the 126 MB L2"}
    return cfg


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------

def time_launches(fn, steps, warmup, stream_sync):
    """CUDA events on the current stream around `steps` back-to-back calls; returns total ms."""
    import torch
    for _ in range(warmup):
        fn()
    stream_sync()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        fn()
    stop.record()
    stop.synchronize()
    return start.elapsed_time(stop)


def reference_streams(steps=10, warmup=3):
    """A plain device copy and a write-only fill of 2 GiB, timed in this run on this GPU (library kernels, context for the
    roofline denominator only: the measured copy bandwidth of MEASURED_PEAKS.json stays the peak the fraction uses)."""
    import torch
    n = 1 << 29  # elements of 4 bytes
    src = torch.empty(n, dtype=torch.float32, device="cuda")
    dst = torch.empty(n, dtype=torch.float32, device="cuda")
    src.fill_(1.0)
    ms_copy = time_launches(lambda: dst.copy_(src), steps, warmup, torch.cuda.synchronize) / steps
    ms_fill = time_launches(lambda: dst.fill_(3.0), steps, warmup, torch.cuda.synchronize) / steps
    del src, dst
    return {"copy_gbs": 2 * 4 * n / (ms_copy * 1e-3) / 1e9, "write_only_gbs": 4 * n / (ms_fill * 1e-3) / 1e9,
            "bytes": 4 * n, "note": "torch copy_ (read + write) and fill_ (write only) of 2 GiB of float32, after the timed region"}


def secondary_config(binding, inputs, name, peaks, steps=20, warmup=3):
    """Short kernel-only measurement of one of the other configurations (reported, not the headline).  For the row
    Softmax the two recomputing forms of Section VI-A are timed on the same buffers as well (``forms_ms``)."""
    import torch
    w = inputs.WORKLOADS[name]
    if w.kind == "rows":
        S = torch.empty((w.rows, w.cols), dtype=torch.float32, device="cuda")
        blk = 4096
        for r0 in range(0, w.rows, blk):
            S[r0:r0 + blk].copy_(torch.from_numpy(inputs.make_scores(w, r0, r0 + blk)))
        P = torch.empty((w.rows, w.cols), dtype=torch.bfloat16, device="cuda")
        fn = lambda: binding.softmax_rows(S, P=P)  # noqa: E731
    else:
        q, k = inputs.make_qk(w)
        Q = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).reshape(w.B, w.H, w.N, w.d).cuda()
        K = torch.from_numpy(k.view(np.int16)).view(torch.bfloat16).reshape(w.B, w.H, w.N, w.d).cuda()
        P = torch.empty((w.B, w.H, w.N, w.N), dtype=torch.bfloat16 if w.p_dtype == "bf16" else torch.float32,
                        device="cuda")
        fn = lambda: binding.attnw_fused(Q, K, w.scale, P=P)  # noqa: E731
    ms = time_launches(fn, steps, warmup, torch.cuda.synchronize) / steps
    forms = None
    if w.kind == "rows":
        forms = {"caching": ms}
        for form in ("recomputing_registers", "recomputing"):
            binding.set_rows_variant(form)
            try:
                forms[form] = time_launches(fn, steps, warmup, torch.cuda.synchronize) / steps
            finally:
                binding.set_rows_variant("auto")
    bytes_alg = w.in_bytes + w.p_bytes
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_flop = w.flops / (peaks["bf16_tflops"] * 1e12)
    out = {"elements_per_s": w.elements / (ms * 1e-3), "ms": ms, "achieved_gbs": bytes_alg / (ms * 1e-3) / 1e9,
           "roofline_frac": max(t_hbm, t_flop) / (ms * 1e-3), "bound": "hbm" if t_hbm >= t_flop else "tensor",
           "steps": steps}
    if forms:
        out["forms_ms"] = forms
    return out


def long_rows_config(binding, peaks, steps=10, warmup=3):
    """Row Softmax on long rows (the row-length axis of the paper's per-element runtime figure): 2^28 float32 scores
    drawn on the device (values N(0, 3^2) as in c4; a timing-only line, parity is the tests' job) in rows of 32768 to
    262144 columns; picoseconds per element against the copy roofline (6 bytes per element)."""
    import torch
    total = 1 << 28
    g = torch.Generator(device="cuda")
    g.manual_seed(4)
    S = torch.empty(total, dtype=torch.float32, device="cuda")
    S.normal_(0.0, 3.0, generator=g)
    P = torch.empty(total, dtype=torch.bfloat16, device="cuda")
    roof_ps = 6.0 / (peaks["hbm_gbs"] * 1e9) * 1e12
    out = {"elements_per_launch": total, "roofline_ps_per_element": roof_ps, "steps": steps}
    for cols in (32768, 65536, 131072, 262144):
        s2, p2 = S.view(total // cols, cols), P.view(total // cols, cols)
        ms = time_launches(lambda: binding.softmax_rows(s2, P=p2), steps, warmup, torch.cuda.synchronize) / steps
        ps = ms * 1e-3 / total * 1e12
        out[str(cols)] = {"ms": ms, "ps_per_element": ps, "roofline_frac": roof_ps / ps}
    del S, P
    return out


def attention_config(binding, inputs, name, peaks, steps=20, warmup=3):
    """Short kernel-only measurement of attn_fused (the product with V, Section IV) on the shape of one of the
    configurations, with V drawn like K on its own stream (reported beside the headline, not part of it)."""
    import torch
    w = inputs.WORKLOADS[name]
    q, k = inputs.make_qk(w)
    v = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 100, w.B * w.H * w.N * w.d, 1.0)
    as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).reshape(w.B, w.H, w.N, w.d).cuda()  # noqa: E731
    Q, K, V = as_t(q), as_t(k), as_t(v)
    O = torch.empty_like(Q)
    ms = time_launches(lambda: binding.attn_fused(Q, K, V, w.scale, O=O), steps, warmup, torch.cuda.synchronize) / steps
    flops = 2.0 * w.flops                       # Q K^T and P V, 2 N^2 d multiply-adds each per head
    bytes_alg = 4 * w.B * w.H * w.N * w.d * 2   # Q, K, V read once, O written once
    t_flop = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    return {"op": "attn_fused: O = Softmax(scale Q K^T) V, bf16", "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
            "roofline_frac": max(t_hbm, t_flop) / (ms * 1e-3), "bound": "tensor" if t_flop >= t_hbm else "hbm",
            "peak_tflops": peaks["bf16_tflops"], "algorithmic_flops": flops, "steps": steps}


def projection_inputs(inputs, w, B):
    """X [B, N, d_model] ~ N(0, 1) and Wq, Wk [H, d, d_model] ~ N(0, 1/d_model) with d_model = H * d: the inputs that
    produce queries and keys distributed like the headline workload's (bf16 bit patterns, seeded, on their own streams)."""
    dm = w.H * w.d
    x = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 200, B * w.N * dm, 1.0)
    wq = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 201, w.H * w.d * dm, dm ** -0.5)
    wk = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 202, w.H * w.d * dm, dm ** -0.5)
    return x, wq, wk, dm


def projection_config(binding, inputs, name, peaks, steps=20, warmup=3):
    """Short kernel-only measurement of attnw_project_qk (queries and keys from the inputs, Section IV) for the shape of
    one of the configurations with d_model = H * d (reported beside the headline, not part of it)."""
    import torch
    w = inputs.WORKLOADS[name]
    x, wq, wk, dm = projection_inputs(inputs, w, w.B)
    as_t = lambda a, shape: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).reshape(shape).cuda()  # noqa: E731
    X, Wq, Wk = as_t(x, (w.B, w.N, dm)), as_t(wq, (w.H, w.d, dm)), as_t(wk, (w.H, w.d, dm))
    Q = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.bfloat16, device="cuda")
    K = torch.empty_like(Q)
    ms = time_launches(lambda: binding.project_qk(X, Wq, Wk, Q=Q, K=K), steps, warmup, torch.cuda.synchronize) / steps
    flops = 2.0 * w.B * w.N * dm * 2 * w.H * w.d      # two products of [B N, d_model] with [d_model, H d]
    bytes_alg = (w.B * w.N * dm + 2 * w.H * w.d * dm + 2 * w.B * w.H * w.N * w.d) * 2
    t_flop = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    return {"op": f"attnw_project_qk: Q, K = X Wq, X Wk, bf16, d_model={dm}", "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
            "roofline_frac": max(t_hbm, t_flop) / (ms * 1e-3), "bound": "tensor" if t_flop >= t_hbm else "hbm",
            "peak_tflops": peaks["bf16_tflops"], "algorithmic_flops": flops, "steps": steps}


def run_profile_case(args):
    """A reduced case of one kernel for profiler captures (`--profile fused|rows`): the same kernel and
    tile configuration as the headline launch on inputs that still exceed the L2 but hold well under a
    GB on the device.  Prints one JSON line marked as a profile run; never a benchmark value."""
    import torch
    from paper_2407_13885_b200 import binding, inputs
    torch.cuda.set_device(0)
    binding.set_fused_variant(args.variant)
    if args.profile == "fused":
        base = inputs.WORKLOADS[args.workload]
        heads = max(1, min(base.B * base.H, (512 << 20) // (base.N * base.N * 2)))
        w = inputs.Workload(base.name + "-reduced", "fused", B=1, H=heads, N=base.N, d=base.d, sigma=base.sigma,
                            scale=base.scale, p_dtype=base.p_dtype, cfg_id=base.cfg_id)
        q, k = inputs.make_qk(w)
        Q = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).reshape(1, heads, w.N, w.d).cuda()
        K = torch.from_numpy(k.view(np.int16)).view(torch.bfloat16).reshape(1, heads, w.N, w.d).cuda()
        P = torch.empty((1, heads, w.N, w.N), dtype=torch.bfloat16, device="cuda")
        fn = lambda: binding.attnw_fused(Q, K, w.scale, P=P)  # noqa: E731
        desc = f"fused B=1 H={heads} N={w.N} d={w.d} (P {w.p_bytes >> 20} MiB)"
    elif args.profile == "attention":
        base = inputs.WORKLOADS[args.workload]
        heads = 16
        w = inputs.Workload(base.name + "-attention-reduced", "fused", B=1, H=heads, N=base.N, d=base.d, sigma=base.sigma,
                            scale=base.scale, p_dtype=base.p_dtype, cfg_id=base.cfg_id)
        q, k = inputs.make_qk(w)
        v = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 100, heads * w.N * w.d, 1.0)
        as_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).reshape(1, heads, w.N, w.d).cuda()  # noqa: E731
        Q, K, V = as_t(q), as_t(k), as_t(v)
        O = torch.empty_like(Q)
        fn = lambda: binding.attn_fused(Q, K, V, w.scale, O=O)  # noqa: E731
        desc = f"attn_fused B=1 H={heads} N={w.N} d={w.d}"
    elif args.profile == "project":
        w = inputs.WORKLOADS[args.workload]
        x, wq, wk, dm = projection_inputs(inputs, w, 1)   # one batch entry of the configuration
        as_t = lambda a, shape: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).reshape(shape).cuda()  # noqa: E731
        X, Wq, Wk = as_t(x, (1, w.N, dm)), as_t(wq, (w.H, w.d, dm)), as_t(wk, (w.H, w.d, dm))
        Q = torch.empty((1, w.H, w.N, w.d), dtype=torch.bfloat16, device="cuda")
        K = torch.empty_like(Q)
        fn = lambda: binding.project_qk(X, Wq, Wk, Q=Q, K=K)  # noqa: E731
        desc = f"attnw_project_qk B=1 N={w.N} d_model={dm} H={w.H} d={w.d}"
    elif args.profile in ("rows_long", "rows_cluster"):
        # rows beyond the register tier: kept in the shared memory of a cluster of two CTAs (32768 columns), or in the
        # registers of a cluster of eight (131072 columns)
        rows, cols = (4096, 32768) if args.profile == "rows_long" else (1024, 131072)
        w = inputs.Workload("rows-long", "rows", rows=rows, cols=cols, sigma=3.0, cfg_id=4)
        S = torch.from_numpy(inputs.make_scores(w, 0, rows)).cuda()
        P = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
        fn = lambda: binding.softmax_rows(S, P=P)  # noqa: E731
        desc = f"softmax_rows rows={rows} cols={cols} (S {w.in_bytes >> 20} MiB, P {w.p_bytes >> 20} MiB)"
    else:
        base = inputs.WORKLOADS["c4"]
        rows = 8192
        S = torch.from_numpy(inputs.make_scores(base, 0, rows)).cuda()
        P = torch.empty((rows, base.cols), dtype=torch.bfloat16, device="cuda")
        w = inputs.Workload("c4-reduced", "rows", rows=rows, cols=base.cols, sigma=base.sigma, cfg_id=4)
        fn = lambda: binding.softmax_rows(S, P=P)  # noqa: E731
        desc = f"softmax_rows rows={rows} cols={base.cols} (S {w.in_bytes >> 20} MiB, P {w.p_bytes >> 20} MiB)"
    ms = time_launches(fn, args.steps, max(args.warmup, 1), torch.cuda.synchronize) / args.steps
    print(json.dumps({"profile_run": True, "case": desc, "ms_per_launch": ms,
                      "algorithmic_bytes_per_launch": w.in_bytes + w.p_bytes,
                      "achieved_gbs": (w.in_bytes + w.p_bytes) / (ms * 1e-3) / 1e9, "steps": args.steps}))
    return 0


def headline_kernel(variant: str, w):
    """(description, key into profiles/ncu_traffic.json) of the kernel `attnw_fused` runs for this workload."""
    bf16 = w.p_dtype == "bf16"
    if variant == "gridrow" or (variant == "auto" and bf16 and w.N <= 4096):
        return (f"attnw_gridrow_kernel<{w.d}> (groups of {(w.N + 255) // 256} CTAs on a cooperative grid, one launch)",
                f"attnw_gridrow_d{w.d}_N{w.N}")
    if variant == "resident" and bf16 and w.N <= 8192:
        return (f"attnw_resident_kernel<{w.d}> (SRAM-resident, clusters of {(w.N + 511) // 512})",
                f"attnw_resident_d{w.d}_N{w.N}")
    return (f"attnw_fused_kernel<{w.d}, {w.p_dtype}> (two-pass)", f"attnw_fused_d{w.d}_N{w.N}")


def run_ours(args):
    import torch
    from paper_2407_13885_b200 import binding, inputs  # raises if libattnw.so is missing: no fallback

    rank, world, local = dist_env()
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run (one rank per GPU)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    w = inputs.WORKLOADS[args.workload]
    peaks = load_peaks()
    binding.set_fused_variant(args.variant)

    # seeded inputs: every rank draws its own replica of the workload (weak scaling, the default), or its slice of the
    # heads of ONE workload (--scaling strong); either way no data crosses ranks
    h_begin, h_end, seed = inputs.rank_heads(w, rank, world, args.scaling)
    n_heads = h_end - h_begin
    if n_heads < 1:
        raise SystemExit(f"rank {rank} owns no head of {w.name}: fewer heads than ranks")
    q, k = inputs.make_qk(w, h_begin, h_end, seed=seed)
    if args.scaling == "strong":
        w_local = inputs.Workload(w.name, "fused", B=1, H=n_heads, N=w.N, d=w.d, sigma=w.sigma, scale=w.scale,
                                  p_dtype=w.p_dtype, cfg_id=w.cfg_id)
    else:
        w_local = w
    w_total_elements = w.elements if args.scaling == "strong" else world * w.elements
    w_whole, w = w, w_local
    shape = (w.B, w.H, w.N, w.d)
    Qh = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).reshape(shape).pin_memory()
    Kh = torch.from_numpy(k.view(np.int16)).view(torch.bfloat16).reshape(shape).pin_memory()
    Q, K = Qh.cuda(), Kh.cuda()
    p_dtype = torch.bfloat16 if w.p_dtype == "bf16" else torch.float32
    P = torch.empty((w.B, w.H, w.N, w.N), dtype=p_dtype, device="cuda")

    def step():
        binding.attnw_fused(Q, K, w.scale, P=P)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    binding.launch_count(reset=True)
    # one event after every step (launches stay back to back; nothing synchronises inside the timed region)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    marks[0].record()
    for i in range(args.steps):
        step()
        marks[i + 1].record()
    torch.cuda.synchronize()
    barrier()
    launches = binding.launch_count()
    sampler.halt.set()
    sampler.join()
    elapsed_ms = marks[0].elapsed_time(marks[-1])
    per_step = np.array([marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)])
    status = binding.query_status()
    if status != 0:
        raise SystemExit(f"device status word {status:#x}: a bounded wait gave up; timing is invalid")
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([elapsed_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
        lt = torch.tensor([launches], dtype=torch.int64, device="cuda")
        dist.all_reduce(lt, op=dist.ReduceOp.SUM)
        launches = int(lt.item())
    ms_per_step = elapsed_ms / args.steps
    value = w_total_elements / (ms_per_step * 1e-3)

    # ---- end to end through the host-buffer C-ABI call ----
    e2e = None
    if not args.no_e2e:
        Ph = torch.empty((w.B, w.H, w.N, w.N), dtype=p_dtype).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        binding.host_attnw_fused(Qh, Kh, w.scale, Ph)  # warm-up: allocates the staging buffers
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            binding.host_attnw_fused(Qh, Kh, w.scale, Ph)  # returns when P is complete in host memory
        dt = time.perf_counter() - t0
        barrier()
        if world > 1:
            import torch.distributed as dist
            t = torch.tensor([dt], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        e2e = {"value": w_total_elements * e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": w.in_bytes, "d2h_bytes_per_step": w.p_bytes,
               "steps": e2e_steps, "ms_per_step": 1e3 * dt / e2e_steps,
               "note": "attnw_fused_host: pinned host Q,K -> device, kernel, P -> pinned host, pipelined over "
                       "groups of heads on two streams; wall clock around the blocking call"}
        binding.host_release()
        del Ph

    if rank != 0:
        return 0

    bytes_alg = w.in_bytes + w.p_bytes
    kernel_s = ms_per_step * 1e-3
    achieved = bytes_alg / kernel_s / 1e9
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_flop = w.flops / (peaks["bf16_tflops"] * 1e12)
    kernel_name, kernel_key = headline_kernel(args.variant, w)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"],
                "traffic": measured_traffic(kernel_key, w.B * w.H),
                "traffic_source": f"profiles/ncu_traffic.json[{kernel_key}] x {w.B * w.H} heads",
                "peak_source": f"of {peaks['source']}",
                "algorithmic_bytes_per_launch": bytes_alg,
                "roofline_time_us": 1e6 * max(t_hbm, t_flop), "kernel_time_us": 1e6 * kernel_s,
                "time_frac_of_roofline": max(t_hbm, t_flop) / kernel_s,
                "tensor_time_us_at_burst_peak": 1e6 * t_flop,
                "kernel": kernel_name}
    step_ms = {"median": float(np.median(per_step)), "min": float(per_step.min()), "max": float(per_step.max()),
               "mean": float(per_step.mean()),
               "note": "one CUDA event after every launch of the timed region (rank 0); launches back to back"}
    roofline["frac_at_median_step"] = bytes_alg / (step_ms["median"] * 1e-3) / 1e9 / peaks["hbm_gbs"]

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": args.scaling, "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(w_whole, world, args.scaling), "clocks": sampler.summary(), "e2e": e2e,
            "gpu_launches": launches, "roofline": roofline, "step_ms": step_ms}

    if not args.no_sustained and world == 1:
        # A multi-second loop of the same launch: the chip settles at its power limit (about 1.45-1.55 GHz
        # instead of the 1.9 GHz of a short burst), which the timed region above is too short to reach.
        t_end = time.perf_counter() + args.sustained_seconds
        n_loop, ms_loop = 0, 0.0
        while time.perf_counter() < t_end:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(100):
                step()
            b.record()
            torch.cuda.synchronize()
            ms_loop = a.elapsed_time(b) / 100
            n_loop += 100
        line["sustained"] = {"ms_per_step": ms_loop, "value": w.elements / (ms_loop * 1e-3), "unit": UNIT,
                             "roofline_frac": bytes_alg / (ms_loop * 1e-3) / 1e9 / peaks["hbm_gbs"],
                             "launches": n_loop,
                             "note": "last 100 of a %.0f s back-to-back loop; power-capped clocks" % args.sustained_seconds}
        roofline["frac_sustained"] = line["sustained"]["roofline_frac"]
    if not args.no_cpu_baseline:
        _, info, _, _ = oracle_sample_rate(w, args.cpu_seconds)
        info["paper_cpu_c4"] = paper_cpu_rows_line()
        line["cpu_baseline"] = info
    if not args.no_secondary and world == 1:
        del P, Q, K
        torch.cuda.empty_cache()
        line["reference_streams"] = reference_streams()
        # the same launch against the write-only stream measured in this run (P is 94 % of the bytes and all writes)
        roofline["frac_of_write_only_stream"] = achieved / line["reference_streams"]["write_only_gbs"]
        torch.cuda.empty_cache()
        other = {}
        for name in ("c4", "c5", "c2"):
            other[name] = secondary_config(binding, inputs, name, peaks)
            torch.cuda.empty_cache()
        other["softmax_rows_long"] = long_rows_config(binding, peaks)
        torch.cuda.empty_cache()
        other["attention_c3"] = attention_config(binding, inputs, "c3", peaks)
        torch.cuda.empty_cache()
        other["project_qk_c3"] = projection_config(binding, inputs, "c3", peaks)
        torch.cuda.empty_cache()
        line["other_configs"] = other
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=HEADLINE, choices=["c2", "c3", "c5"])
    ap.add_argument("--scaling", choices=["weak", "strong"], default="weak",
                    help="weak: every rank runs a whole replica (default); strong: the heads of ONE workload are dealt out")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--sustained-seconds", type=float, default=2.0)
    ap.add_argument("--variant", choices=["auto", "two_pass", "resident", "gridrow"], default="auto",
                    help="kernel behind attnw_fused (see attnw_set_fused_variant)")
    ap.add_argument("--profile", choices=["fused", "rows", "rows_long", "rows_cluster", "attention", "project"], default=None,
                    help="run a reduced case of one kernel for an ncu capture instead of the benchmark")
    ap.add_argument("--timeline", action="store_true",
                    help="per-phase cycle table of the headline kernel from an instrumented build (see timeline.py)")
    args = ap.parse_args()
    if args.timeline:
        from paper_2407_13885_b200 import timeline
        return timeline.main([])
    if args.impl == "reference":
        return run_reference(args)
    if args.profile:
        return run_profile_case(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
