"""softmax_rows on the GPU against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, assert_close_to_oracle, assert_guards_intact, guarded_empty
from paper_2407_13885_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def attnw():
    from paper_2407_13885_b200 import binding
    return binding


# every kernel tier and both sides of each tier boundary, with ragged tails
SHAPES = [(1, 4), (3, 8), (33, 36), (257, 100), (64, 128), (5, 132), (40, 260), (17, 1000), (9, 1024),
          (7, 1028), (6, 2052), (5, 4096), (4, 4100), (3, 8192), (3, 8196), (2, 16384), (2, 16388),
          (2, 32768), (3, 32772), (2, 70000), (600, 512),
          # beyond 32768 columns the rows live in the registers of a cluster of 3 to 16 CTAs (any size, ragged last slice,
          # more rows than clusters, its last column count), then the two-read tier
          (5, 40000), (3, 49152), (2, 100000), (1, 196608), (300, 33000), (1, 393216), (2, 393220), (40, 98308),
          (9, 65536), (4, 81924), (150, 57348), (3, 180228), (3, 262144), (2, 262148), (33, 245764)]


@pytest.mark.parametrize("rows,cols", SHAPES)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_rows_match_oracle(attnw, rows, cols, dtype):
    S = inputs.normal_f32(11, rows * 131 + cols, rows * cols, 3.0).reshape(rows, cols)
    raw, P, g = guarded_empty((rows, cols), dtype)
    attnw.softmax_rows(torch.from_numpy(S).cuda(), P=P)
    torch.cuda.synchronize()
    assert_guards_intact(raw, g)
    assert_close_to_oracle(P, oracle.softmax_rows(S), f"rows={rows} cols={cols}")
    assert attnw.query_status() == 0


@pytest.mark.parametrize("rows,cols", [(3, 8), (257, 100), (40, 260), (9, 1024), (5, 4096), (3, 8196), (2, 32768), (600, 512)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("form", ["recomputing", "recomputing_registers"])
def test_recomputing_form_matches_oracle(attnw, rows, cols, dtype, form):
    # the "recomputing" form of Section VI-A on row lengths the default serves from registers
    S = inputs.normal_f32(11, rows * 137 + cols, rows * cols, 3.0).reshape(rows, cols)
    raw, P, g = guarded_empty((rows, cols), dtype)
    attnw.set_rows_variant(form)
    try:
        attnw.softmax_rows(torch.from_numpy(S).cuda(), P=P)
        torch.cuda.synchronize()
    finally:
        attnw.set_rows_variant("auto")
    assert_guards_intact(raw, g)
    assert_close_to_oracle(P, oracle.softmax_rows(S), f"recomputing rows={rows} cols={cols}")
    assert attnw.query_status() == 0


@pytest.mark.parametrize("rows,cols", [(2, 70000), (2, 100000), (1, 196608), (40, 98308), (1, 393216)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_cluster_cached_rows_match_oracle(attnw, rows, cols, dtype):
    # the caching form on request: the row lives in the shared memory of a cluster of 4, 8 or 16 CTAs
    S = inputs.normal_f32(11, rows * 139 + cols, rows * cols, 3.0).reshape(rows, cols)
    raw, P, g = guarded_empty((rows, cols), dtype)
    attnw.set_rows_variant("caching")
    try:
        attnw.softmax_rows(torch.from_numpy(S).cuda(), P=P)
        torch.cuda.synchronize()
    finally:
        attnw.set_rows_variant("auto")
    assert_guards_intact(raw, g)
    assert_close_to_oracle(P, oracle.softmax_rows(S), f"cluster-cached rows={rows} cols={cols}")
    assert attnw.query_status() == 0


def test_caching_only_refuses_rows_beyond_the_on_chip_tiers(attnw):
    S = torch.zeros((1, 393220), dtype=torch.float32, device="cuda")
    attnw.set_rows_variant("caching")
    try:
        with pytest.raises(attnw.AttnwError) as e:
            attnw.softmax_rows(S)
        assert e.value.code == 4
        P = attnw.softmax_rows(S[:, :40000].contiguous())   # kept in shared memory: still the caching form
        torch.cuda.synchronize()
        assert bool((P.float() == 1.0 / 40000).all()) or float((P.float() - 1.0 / 40000).abs().max()) < 1e-7
    finally:
        attnw.set_rows_variant("auto")


def test_in_place_f32(attnw):
    S = inputs.normal_f32(12, 1, 50 * 4096, 3.0).reshape(50, 4096)
    buf = torch.from_numpy(S).cuda()
    attnw.softmax_rows(buf, P=buf)
    torch.cuda.synchronize()
    assert_close_to_oracle(buf, oracle.softmax_rows(S), "in place")
    S2 = inputs.normal_f32(12, 2, 2 * 70000, 3.0).reshape(2, 70000)  # streaming tier in place
    buf = torch.from_numpy(S2).cuda()
    attnw.softmax_rows(buf, P=buf)
    torch.cuda.synchronize()
    assert_close_to_oracle(buf, oracle.softmax_rows(S2), "in place, streaming tier")


def test_large_logits_and_constant_rows(attnw):
    S = np.zeros((4, 2048), dtype=np.float32)
    S[0, :] = 1.0e4
    S[0, 5] = -1.0e4
    S[1, :] = -3.0e4
    S[2, 100] = 800.0
    S[3, :] = inputs.normal_f32(13, 3, 2048, 30.0)
    for dtype in (torch.bfloat16, torch.float32):
        P = attnw.softmax_rows(torch.from_numpy(S).cuda(), out_dtype=dtype)
        torch.cuda.synchronize()
        assert_close_to_oracle(P, oracle.softmax_rows(S), "large logits")
    # a constant row of a power-of-two length is exactly uniform
    assert bool((P[1] == 1.0 / 2048).all())


def test_config_c4_full_size(attnw):
    """rows=32768, cols=8192 fp32 -> bf16, the launch the benchmark times; oracle on every row."""
    w = inputs.WORKLOADS["c4"]
    P = torch.empty((w.rows, w.cols), dtype=torch.bfloat16, device="cuda")
    P.view(torch.int16).fill_(-1)  # NaN bit pattern: an element left unwritten would show
    S_dev = torch.empty((w.rows, w.cols), dtype=torch.float32, device="cuda")
    block = 4096
    for r0 in range(0, w.rows, block):
        S_dev[r0:r0 + block].copy_(torch.from_numpy(inputs.make_scores(w, r0, r0 + block)))
    attnw.softmax_rows(S_dev, P=P)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    assert not bool(torch.isnan(P).any())
    worst = 0.0
    for r0 in range(0, w.rows, block):
        ref = oracle.softmax_rows(inputs.make_scores(w, r0, r0 + block))
        err, _ = assert_close_to_oracle(P[r0:r0 + block], ref, f"c4 rows {r0}..")
        worst = max(worst, err)
    assert worst <= TOL[torch.bfloat16]["abs"]


def test_bad_arguments_on_device(attnw):
    S = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(attnw.AttnwError) as e:
        attnw.softmax_rows(S[:, :6].contiguous())
    assert e.value.code == 3
    alias = S.view(torch.bfloat16).reshape(-1)[:32].view(4, 8)  # a bf16 output inside the input
    with pytest.raises(attnw.AttnwError) as e:
        attnw.softmax_rows(S, P=alias)
    assert e.value.code == 7
