"""Shared pieces of the GPU parity tests: tolerances, conversions, comparison."""
import numpy as np
import torch

from paper_2407_13885_b200 import inputs

# Acceptance tolerances for the CUDA path against the fp64 oracle.
TOL = {
    torch.bfloat16: {"abs": 4e-3, "rowsum": 1e-2},
    torch.float32: {"abs": 2e-5, "rowsum": 1e-5},
}


def bits_to_cuda_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor of the same shape (no rounding)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.bfloat16).to(device)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def assert_close_to_oracle(P_gpu: torch.Tensor, P_ref: np.ndarray, what: str = ""):
    tol = TOL[P_gpu.dtype]
    got = to_f64(P_gpu).reshape(P_ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = float(np.max(np.abs(got - P_ref)))
    assert err <= tol["abs"], f"{what}: max abs err {err:.3e} > {tol['abs']}"
    rs = float(np.max(np.abs(got.sum(-1) - 1.0)))
    assert rs <= tol["rowsum"], f"{what}: row sum off by {rs:.3e} > {tol['rowsum']}"
    assert got.min() >= 0.0 and got.max() <= 1.0 + 1e-6, f"{what}: value outside [0,1]"
    return err, rs


def guarded_empty(shape, dtype, device="cuda", guard_elems=2048):
    """Output tensor carved out of a larger buffer whose margins hold a sentinel and whose body is
    pre-filled with NaN: shows out-of-bounds writes and elements the kernel failed to write."""
    n = int(np.prod(shape))
    raw = torch.empty(n + 2 * guard_elems, dtype=dtype, device=device)
    raw.fill_(-7.0)
    body = raw[guard_elems:guard_elems + n]
    body.fill_(float("nan"))
    return raw, body.view(shape), guard_elems


def assert_guards_intact(raw: torch.Tensor, guard_elems: int):
    assert bool((raw[:guard_elems] == -7.0).all()), "wrote before the output buffer"
    assert bool((raw[-guard_elems:] == -7.0).all()), "wrote past the output buffer"


def small_fused_inputs(B, H, N, d, sigma=1.0, stream=1000):
    n = B * H * N * d
    q = inputs.normal_bf16_bits(99, stream, n, sigma).reshape(B, H, N, d)
    k = inputs.normal_bf16_bits(99, stream + 1, n, sigma).reshape(B, H, N, d)
    return q, k
