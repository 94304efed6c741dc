"""attn_fused (Attention(Q, K, V) of Section IV in one kernel) on the GPU against the fp64 oracle, through the C ABI."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import bits_to_cuda_bf16, small_fused_inputs
from paper_2407_13885_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["one_pass", "two_pass"])
def attnw(request):
    from paper_2407_13885_b200 import binding
    binding.set_attn_variant(request.param)
    yield binding
    binding.set_attn_variant("auto")


def rand_v(B, H, N, d, sigma=1.0, stream=900):
    return inputs.normal_bf16_bits(11, stream, B * H * N * d, sigma).reshape(B, H, N, d)


def run_attn(attnw, q, k, v, scale):
    B, H, N, d = q.shape
    # guard rows before and after O: the kernel must write O and nothing else
    raw = torch.full((B * H * N * d + 2 * 4096,), float("nan"), dtype=torch.bfloat16, device="cuda")
    O = raw[4096:4096 + B * H * N * d].view(B, H, N, d)
    attnw.attn_fused(bits_to_cuda_bf16(q), bits_to_cuda_bf16(k), bits_to_cuda_bf16(v), scale, O=O)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    assert bool(torch.isnan(raw[:4096]).all()) and bool(torch.isnan(raw[-4096:]).all())
    return O


def tolerance(v_bits):
    # bf16 keeps 8 significant bits: rounding to nearest moves a value by at most 2^-8 of itself (at the bottom of a
    # binade).  The weights enter the second product rounded to bf16 and sum to one, O is rounded to bf16 and
    # |O| <= max|V|:  |O_gpu - O| <= 2^-8 sum_j p_j |v_j| + 2^-8 |O| <= 2^-7 max|V|, plus float32 dust.
    return 2.0 ** -7 * float(np.abs(inputs.bf16_bits_to_f32(v_bits)).max()) + 1e-5


def tolerance_map(q, k, v, scale, ref, row_ids=None):
    # The same bound per element instead of its maximum: 2^-8 (sum_j p_j |v_j| + |O|), where the first sum is the
    # oracle's attention over the absolute values of V.
    v_abs = inputs.f32_to_bf16_bits(np.abs(inputs.bf16_bits_to_f32(v)))   # |v| is exact in bf16
    mass = oracle.attn(q, k, v_abs, scale, row_ids=row_ids)
    return 2.0 ** -8 * (mass + np.abs(ref)) + 1e-5


SHAPES = [(1, 1, 128, 64), (1, 1, 128, 128), (1, 2, 256, 64), (2, 1, 384, 128), (1, 3, 512, 64), (1, 1, 8, 64),
          (1, 2, 72, 128), (1, 1, 136, 64), (2, 2, 200, 128), (1, 1, 264, 64), (1, 1, 1000, 128), (1, 1, 1160, 64),
          (1, 1, 1, 64), (1, 1, 77, 128)]


@pytest.mark.parametrize("B,H,N,d", SHAPES)
def test_attention_matches_oracle(attnw, B, H, N, d):
    q, k = small_fused_inputs(B, H, N, d, stream=N + d + 3)
    v = rand_v(B, H, N, d, stream=N + d + 5)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    O = run_attn(attnw, q, k, v, scale)
    ref = oracle.attn(q, k, v, scale)
    got = O.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    tol = tolerance_map(q, k, v, scale, ref)
    assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))


@pytest.mark.parametrize("B,H,N,d", [(1, 2, 1024, 128), (2, 2, 513, 64)])
def test_attention_large_logits(attnw, B, H, N, d):
    q, k = small_fused_inputs(B, H, N, d, sigma=4.0, stream=61 + N)
    v = rand_v(B, H, N, d, stream=62 + N)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    O = run_attn(attnw, q, k, v, scale)
    ref = oracle.attn(q, k, v, scale)
    got = O.float().cpu().numpy().astype(np.float64)
    # At sigma = 4 the raw scores reach ~1e3 and the tensor cores' float32 accumulation error of a score,
    # (d/16) * 17 * 2^-24 * max|s|, is no longer dust: dp <= p * scale * ds for every weight of a row, and a
    # perturbed row moves that much weight from some keys to others, so dO <= 2 * scale * ds * max|V| on top.
    s_abs = float(np.max(np.abs(oracle.scores_rows(q, k, np.arange(B * H * N)))))
    v_abs = float(np.abs(inputs.bf16_bits_to_f32(v)).max())
    tol = tolerance_map(q, k, v, scale, ref) + 2.0 * scale * s_abs * (d / 16) * 17 * 2.0 ** -24 * v_abs
    err = np.abs(got - ref)
    assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))


def test_attention_with_row_maxima_that_keep_growing(attnw):
    # Keys whose norm grows with the key index: the running row maximum rises in most key tiles, by more than the
    # 2^8 the one-pass kernel tolerates before it moves a row's offset, so O and the row sums are rescaled often.
    B, H, N, d = 1, 2, 1160, 128
    q, k = small_fused_inputs(B, H, N, d, sigma=2.0, stream=63)
    ramp = (0.25 + 4.0 * np.arange(N, dtype=np.float32) / N).reshape(1, 1, N, 1)
    k = inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(k) * ramp)
    v = rand_v(B, H, N, d, stream=64)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    O = run_attn(attnw, q, k, v, scale)
    ref = oracle.attn(q, k, v, scale)
    got = O.float().cpu().numpy().astype(np.float64)
    s_abs = float(np.max(np.abs(oracle.scores_rows(q, k, np.arange(H * N)))))
    v_abs = float(np.abs(inputs.bf16_bits_to_f32(v)).max())
    tol = tolerance_map(q, k, v, scale, ref) + 2.0 * scale * s_abs * (d / 16) * 17 * 2.0 ** -24 * v_abs  # as above
    err = np.abs(got - ref)
    assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))


def test_attention_of_constant_and_unit_vector_values(attnw):
    # constant V: O is that constant (rows of the weights sum to one)
    q, k = small_fused_inputs(1, 2, 520, 128, stream=71)
    ones = inputs.f32_to_bf16_bits(np.full((1, 2, 520, 128), 1.5, dtype=np.float32))
    O = run_attn(attnw, q, k, ones, 0.09)
    assert float((O.float() - 1.5).abs().max()) <= 1.5 * 2.0 ** -7   # the bound of tolerance() for max|V| = 1.5
    # V[j, c] = 1 where c == j mod d: column c of O is the sum of the weights of keys j = c (mod d) - catches any
    # mix-up of the key and feature axes of V
    N, d = 300, 64
    q, k = small_fused_inputs(1, 1, N, d, stream=72)
    vv = np.zeros((1, 1, N, d), dtype=np.float32)
    for j in range(N):
        vv[0, 0, j, j % d] = 1.0
    O = run_attn(attnw, q, k, inputs.f32_to_bf16_bits(vv), 0.125)[0, 0].float().cpu().numpy().astype(np.float64)
    P = oracle.attnw(q, k, 0.125)[0, 0]
    want = np.stack([P[:, c::d].sum(axis=1) for c in range(d)], axis=1)
    assert np.max(np.abs(O - want)) <= 2.0 ** -7   # tolerance() for max|V| = 1


def test_attention_argument_errors(attnw):
    x = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(attnw.AttnwError) as e:
        attnw.attn_fused(x, x, x, 0.1, O=x)
    assert e.value.code == 7
    y = torch.zeros((1, 1, 128, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(attnw.AttnwError) as e:
        attnw.attn_fused(y, y, y, 0.1)
    assert e.value.code == 4


def test_attention_full_size_sampled(attnw):
    """The launch the benchmark times (B=4, H=32, N=4096, d=128, V drawn like the benchmark's): no element left
    unwritten, every output inside the range of V, and oracle parity on sampled complete rows of every head."""
    w = inputs.WORKLOADS["c3"]
    q, k = inputs.make_qk(w)
    q, k = q.reshape(w.B, w.H, w.N, w.d), k.reshape(w.B, w.H, w.N, w.d)
    v = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 100, w.B * w.H * w.N * w.d, 1.0).reshape(w.B, w.H, w.N, w.d)
    O = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.bfloat16, device="cuda")
    O.view(torch.int16).fill_(-1)  # NaN pattern
    V = bits_to_cuda_bf16(v)
    attnw.attn_fused(bits_to_cuda_bf16(q), bits_to_cuda_bf16(k), V, w.scale, O=O)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    assert not bool(torch.isnan(O).any())
    # a convex combination of the values of its head, up to the rounding the tolerance allows
    v_hi = V.float().amax(dim=2, keepdim=True)
    v_lo = V.float().amin(dim=2, keepdim=True)
    slack = tolerance(v)
    assert bool((O.float() <= v_hi + slack).all()) and bool((O.float() >= v_lo - slack).all())
    rng = np.random.default_rng(3)
    ids = []
    for bh in range(w.B * w.H):
        local = {0, 127, 128, w.N - 129, w.N - 1} | set(rng.integers(0, w.N, size=3).tolist())
        ids += [bh * w.N + i for i in sorted(local)]
    ids = np.array(ids, dtype=np.int64)
    ref = oracle.attn(q, k, v, w.scale, row_ids=ids)
    got = O.view(-1, w.d)[torch.from_numpy(ids).cuda()].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    tol = tolerance_map(q, k, v, w.scale, ref, row_ids=ids)
    assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))
