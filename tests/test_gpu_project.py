"""attnw_project_qk (queries and keys from the inputs, Section IV) on the GPU against the fp64 oracle, through the C ABI."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import bits_to_cuda_bf16
from paper_2407_13885_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def attnw():
    from paper_2407_13885_b200 import binding
    return binding


def rand_xw(B, N, d_model, H, d, stream):
    x = inputs.normal_bf16_bits(13, stream, B * N * d_model, 1.0).reshape(B, N, d_model)
    wq = inputs.normal_bf16_bits(13, stream + 1, H * d * d_model, d_model ** -0.5).reshape(H, d, d_model)
    wk = inputs.normal_bf16_bits(13, stream + 2, H * d * d_model, d_model ** -0.5).reshape(H, d, d_model)
    return x, wq, wk


def run_project(attnw, x, wq, wk):
    B, N, _ = x.shape
    H, d, _ = wq.shape
    n = B * H * N * d
    # guards before and after each output: the kernel must write Q and K and nothing else
    raws = [torch.full((n + 2 * 4096,), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    Q, K = (r[4096:4096 + n].view(B, H, N, d) for r in raws)
    attnw.project_qk(bits_to_cuda_bf16(x), bits_to_cuda_bf16(wq), bits_to_cuda_bf16(wk), Q=Q, K=K)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    for r in raws:
        assert bool(torch.isnan(r[:4096]).all()) and bool(torch.isnan(r[-4096:]).all())
    return Q, K


def check(got: torch.Tensor, ref: np.ndarray, x, w):
    # The result is rounded to bf16: 8 significant bits, so half a unit in the last place is at most 2^-8 of the value
    # (reached at the bottom of a binade).  Before that, float32 accumulation in the tensor cores: every
    # partial sum is bounded by sum_m |x_m w_m| and there are d_model / 16 block additions of up to 17 terms each,
    # so the absolute error is below (d_model / 16 + 17) * 2^-24 * max sum |x||w| - far below the rounding of
    # typical entries, but it is what bounds entries that cancel to nearly zero.
    g = got.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all()
    d_model = x.shape[2]
    ax = np.abs(inputs.bf16_bits_to_f32(x).astype(np.float64))
    aw = np.abs(inputs.bf16_bits_to_f32(w).astype(np.float64))
    mass = float(np.einsum("bnm,hcm->bhnc", ax, aw).max())
    tol = 2.0 ** -8 * np.abs(ref) + (d_model / 16 + 17) * 2.0 ** -24 * mass + 1e-30
    err = np.abs(g - ref)
    assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))


# several row tiles and column tiles, ragged rows, ragged d_model (not a multiple of 64), H*d not a multiple of 256,
# a single row, more than one batch entry
SHAPES = [(1, 256, 64, 2, 128), (1, 128, 128, 1, 64), (2, 300, 192, 3, 64), (1, 1, 64, 1, 128), (1, 520, 328, 5, 64),
          (2, 77, 72, 1, 128), (1, 1024, 512, 4, 128), (3, 130, 256, 6, 64), (1, 257, 8, 2, 64)]


@pytest.mark.parametrize("B,N,d_model,H,d", SHAPES)
def test_projection_matches_oracle(attnw, B, N, d_model, H, d):
    x, wq, wk = rand_xw(B, N, d_model, H, d, stream=N + d_model + 7 * H)
    Q, K = run_project(attnw, x, wq, wk)
    check(Q, oracle.project(x, wq), x, wq)
    check(K, oracle.project(x, wk), x, wk)


def test_projection_with_selector_weights_is_exact(attnw):
    # W[h, c, :] = e_{h*d + c}: head h of Q is columns h*d .. of X, bit for bit; K takes them in reverse order
    B, N, H, d = 2, 200, 3, 64
    d_model = H * d
    x = inputs.normal_bf16_bits(13, 90, B * N * d_model, 1.0).reshape(B, N, d_model)
    wq = np.zeros((H, d, d_model), dtype=np.float32)
    wk = np.zeros((H, d, d_model), dtype=np.float32)
    for h in range(H):
        for c in range(d):
            wq[h, c, h * d + c] = 1.0
            wk[h, c, d_model - 1 - (h * d + c)] = 1.0
    Q, K = run_project(attnw, x, inputs.f32_to_bf16_bits(wq), inputs.f32_to_bf16_bits(wk))
    xq = bits_to_cuda_bf16(x)
    want_q = xq.view(B, N, H, d).permute(0, 2, 1, 3)
    want_k = xq.flip(2).view(B, N, H, d).permute(0, 2, 1, 3)
    assert torch.equal(Q, want_q) and torch.equal(K, want_k)


def test_projection_feeds_the_fused_kernel(attnw):
    # the head-major layout is what attnw_fused reads: chain the two and compare with the oracle fed the SAME bf16 Q, K
    B, N, d_model, H, d = 1, 384, 256, 2, 64
    x, wq, wk = rand_xw(B, N, d_model, H, d, stream=95)
    Q, K = run_project(attnw, x, wq, wk)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    P = attnw.attnw_fused(Q, K, scale)
    torch.cuda.synchronize()
    qb = Q.view(torch.int16).cpu().numpy().view(np.uint16)
    kb = K.view(torch.int16).cpu().numpy().view(np.uint16)
    ref = oracle.attnw(qb, kb, scale)
    assert float(np.max(np.abs(P.float().cpu().numpy().astype(np.float64) - ref))) <= 4e-3


def test_projection_argument_errors(attnw):
    x = torch.zeros((1, 128, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((1, 64, 64), dtype=torch.bfloat16, device="cuda")
    w96 = torch.zeros((1, 96, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(attnw.AttnwError) as e:
        attnw.project_qk(x, w96, w96)
    assert e.value.code == 4
    q = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(attnw.AttnwError) as e:
        attnw.project_qk(x, w, w, Q=q, K=q)
    assert e.value.code == 7


def test_projection_full_size_sampled(attnw):
    """The launch the benchmark times (B=4, N=4096, d_model=4096, H=32, d=128, inputs drawn like the benchmark's): no
    element left unwritten and oracle parity on sampled complete rows of every head of Q and of K."""
    w = inputs.WORKLOADS["c3"]
    dm = w.H * w.d
    x = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 200, w.B * w.N * dm, 1.0).reshape(w.B, w.N, dm)
    wq = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 201, w.H * w.d * dm, dm ** -0.5).reshape(w.H, w.d, dm)
    wk = inputs.normal_bf16_bits(inputs.SEED, 2 * w.cfg_id + 202, w.H * w.d * dm, dm ** -0.5).reshape(w.H, w.d, dm)
    Q = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.bfloat16, device="cuda")
    K = torch.empty_like(Q)
    Q.view(torch.int16).fill_(-1)  # NaN pattern
    K.view(torch.int16).fill_(-1)
    attnw.project_qk(bits_to_cuda_bf16(x), bits_to_cuda_bf16(wq), bits_to_cuda_bf16(wk), Q=Q, K=K)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    assert not bool(torch.isnan(Q).any()) and not bool(torch.isnan(K).any())
    rng = np.random.default_rng(4)
    ids = []
    for bh in range(w.B * w.H):
        local = {0, 255, 256, w.N - 1} | set(rng.integers(0, w.N, size=2).tolist())
        ids += [bh * w.N + i for i in sorted(local)]
    ids = np.array(ids, dtype=np.int64)
    sel = torch.from_numpy(ids).cuda()
    # the bound of check(), with the largest sum |x||w| of the sampled rows
    ax = np.abs(inputs.bf16_bits_to_f32(x).astype(np.float64))
    for got_t, wb in ((Q, wq), (K, wk)):
        ref = oracle.project(x, wb, row_ids=ids)
        got = got_t.view(-1, w.d)[sel].float().cpu().numpy().astype(np.float64)
        aw = np.abs(inputs.bf16_bits_to_f32(wb).astype(np.float64))
        mass = 0.0
        for g in ids[::37]:   # a subset is enough for the bound's scale; the maximum over it is then doubled
            n, h, b = g % w.N, (g // w.N) % w.H, g // (w.N * w.H)
            mass = max(mass, float((aw[h] @ ax[b, n]).max()))
        tol = 2.0 ** -8 * np.abs(ref) + (dm / 16 + 17) * 2.0 ** -24 * (2.0 * mass)
        err = np.abs(got - ref)
        assert np.all(err <= tol), (float(err.max()), float((err / tol).max()))
