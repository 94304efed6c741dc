"""The failure path without harming a GPU: a bounded wait that really runs out (on a barrier nobody arrives on, in a
self-test kernel outside every product path), the sticky status word, its clearing, and recovery."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import assert_close_to_oracle, bits_to_cuda_bf16, small_fused_inputs

pytestmark = pytest.mark.gpu

SELFTEST_SITE = 0x80000000 | 127


@pytest.fixture(scope="module")
def attnw():
    from paper_2407_13885_b200 import binding
    return binding


def test_wait_runs_out_status_is_sticky_then_clears_and_work_resumes(attnw):
    assert attnw.query_status() == 0
    q, k = small_fused_inputs(1, 2, 512, 64, stream=301)
    Q, K = bits_to_cuda_bf16(q), bits_to_cuda_bf16(k)
    scale = float(np.float32(1.0 / math.sqrt(64.0)))
    ref = oracle.attnw(q, k, scale)

    attnw.selftest_wait_timeout(1_000_000)           # about half a millisecond, then the wait gives up
    # launches made between the failure and the query write nothing: every CTA sees the word and leaves
    for variant in ("auto", "two_pass", "resident"):
        P = torch.full((1, 2, 512, 512), float("nan"), dtype=torch.bfloat16, device="cuda")
        attnw.set_fused_variant(variant)
        try:
            attnw.attnw_fused(Q, K, scale, P=P)      # returns OK: it only enqueues
        finally:
            attnw.set_fused_variant("auto")
        torch.cuda.synchronize()
        assert bool(torch.isnan(P).all()), f"{variant}: a launch behind a failure wrote output"
    S = torch.randn(64, 16384, device="cuda")         # shared-memory tier of the row Softmax honours the word too
    Pr = torch.full((64, 16384), float("nan"), dtype=torch.bfloat16, device="cuda")
    attnw.softmax_rows(S, P=Pr)
    torch.cuda.synchronize()
    assert bool(torch.isnan(Pr).all())
    Sc = torch.randn(8, 65536, device="cuda")          # ... and so does the cluster tier (registers of four CTAs)
    Pc = torch.full((8, 65536), float("nan"), dtype=torch.bfloat16, device="cuda")
    attnw.softmax_rows(Sc, P=Pc)
    torch.cuda.synchronize()
    assert bool(torch.isnan(Pc).all())

    # the query reports the failure with the site of the wait, once
    word = attnw.query_status()
    assert word == SELFTEST_SITE, hex(word)
    assert attnw.query_status() == 0

    # and the library works again
    for variant in ("auto", "two_pass", "resident"):
        P = torch.full((1, 2, 512, 512), float("nan"), dtype=torch.bfloat16, device="cuda")
        attnw.set_fused_variant(variant)
        try:
            attnw.attnw_fused(Q, K, scale, P=P)
        finally:
            attnw.set_fused_variant("auto")
        torch.cuda.synchronize()
        assert_close_to_oracle(P, ref, f"{variant} after the status was cleared")
    attnw.softmax_rows(Sc, P=Pc)
    torch.cuda.synchronize()
    assert_close_to_oracle(Pc, oracle.softmax_rows(Sc.cpu().numpy()), "cluster tier after the status was cleared")
    assert attnw.query_status() == 0


def test_host_call_reports_and_clears_a_recorded_failure(attnw):
    q, k = small_fused_inputs(1, 1, 256, 64, stream=303)
    Qh = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).pin_memory()
    Kh = torch.from_numpy(k.view(np.int16)).view(torch.bfloat16).pin_memory()
    Ph = torch.empty((1, 1, 256, 256), dtype=torch.bfloat16).pin_memory()
    attnw.selftest_wait_timeout(200_000)
    with pytest.raises(attnw.AttnwError) as e:       # the host call synchronises, so it can and does report it
        attnw.host_attnw_fused(Qh, Kh, 0.125, Ph)
    assert e.value.code == 6
    assert attnw.query_status() == 0                  # ... and has cleared it
    attnw.host_attnw_fused(Qh, Kh, 0.125, Ph)
    assert np.max(np.abs(Ph.to(torch.float64).numpy() - oracle.attnw(q, k, 0.125))) <= 4e-3
    attnw.host_release()


def test_selftest_rejects_limits_out_of_range(attnw):
    for bad in (0, -5, 3_000_000_000):
        with pytest.raises(attnw.AttnwError) as e:
            attnw.selftest_wait_timeout(bad)
        assert e.value.code == 2
    assert attnw.query_status() == 0
