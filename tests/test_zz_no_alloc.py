"""attnw_fused_noalloc, the entry point for callers that cannot allocate device memory (a pool owns the GPU's memory,
or the call sits where cudaMalloc's lock and implicit synchronisation are not acceptable): called through the C ABI,
twice in a row - the second call finds the library's built-in exchange array as the first one left it - and compared
with what attnw_fused produces for the same inputs.  Collected last on purpose: a run that stops at the first failure
has then already run every other test."""
import math

import numpy as np
import pytest
import torch

from helpers import TOL, bits_to_cuda_bf16, small_fused_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def attnw():
    from paper_2407_13885_b200 import binding
    return binding


@pytest.mark.parametrize("B,H,N,d", [(1, 3, 1160, 64), (2, 4, 4096, 128)])
def test_noalloc_matches_attnw_fused_on_two_calls_in_a_row(attnw, B, H, N, d):
    q, k = small_fused_inputs(B, H, N, d, stream=900 + N)
    Q, K = bits_to_cuda_bf16(q), bits_to_cuda_bf16(k)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    ref = attnw.attnw_fused(Q, K, scale).float()          # the existing entry point
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
    for call in range(2):
        P = torch.full((B, H, N, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        lib_rc = attnw.lib.attnw_fused_noalloc(Q.data_ptr(), K.data_ptr(), P.data_ptr(), B, H, N, d, scale, None)
        assert lib_rc == 0
        torch.cuda.synchronize()
        assert attnw.query_status() == 0
        got = P.float()
        assert bool(torch.isfinite(got).all()), f"call {call}: an element was not written"
        err = float((got - ref).abs().max())
        assert err <= TOL[torch.bfloat16]["abs"], f"call {call}: differs from attnw_fused by {err:.3e}"
        assert float((got.double().sum(-1) - 1.0).abs().max()) <= TOL[torch.bfloat16]["rowsum"]


def test_noalloc_refuses_what_it_cannot_serve(attnw):
    big = torch.zeros((1, 1, 4104, 64), dtype=torch.bfloat16, device="cuda")    # more keys than one group holds
    P = torch.empty((1, 1, 4104, 4104), dtype=torch.bfloat16, device="cuda")
    assert attnw.lib.attnw_fused_noalloc(big.data_ptr(), big.data_ptr(), P.data_ptr(), 1, 1, 4104, 64, 0.1, None) == 4
    small = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    Ps = torch.empty((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    assert attnw.lib.attnw_fused_noalloc(None, small.data_ptr(), Ps.data_ptr(), 1, 1, 128, 64, 0.1, None) == 1
    assert attnw.lib.attnw_fused_noalloc(small.data_ptr(), small.data_ptr(), Ps.data_ptr(), 1, 1, 128, 64, -1.0, None) == 2
    with pytest.raises(attnw.AttnwError):
        attnw.attnw_fused_noalloc(big, big, 0.1)
    torch.cuda.synchronize()
    assert attnw.query_status() == 0
