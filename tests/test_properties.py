"""Property tests (hypothesis) of the oracle and of the partition rule: what the definition fixes for ANY input."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2407_13885_b200 import inputs

finite = st.floats(min_value=-50.0, max_value=50.0, allow_nan=False, allow_infinity=False, width=32)


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 5), st.integers(1, 40), st.data())
def test_softmax_rows_invariants(rows, cols, data):
    Z = np.array(data.draw(st.lists(finite, min_size=rows * cols, max_size=rows * cols)), dtype=np.float32).reshape(rows, cols)
    P = oracle.softmax_rows(Z)
    assert P.shape == (rows, cols) and np.all(P >= 0.0) and np.all(P <= 1.0)
    assert np.max(np.abs(P.sum(-1) - 1.0)) <= 1e-12
    shift = np.float32(data.draw(st.integers(-8, 8)))                      # Eq. 1: a common shift of a row changes nothing
    Ps = oracle.softmax_rows((Z.astype(np.float64) + float(shift)).astype(np.float32)) if np.all(
        (Z + shift).astype(np.float32) - shift == Z) else P
    assert np.max(np.abs(Ps - P)) <= 1e-12
    perm = np.array(data.draw(st.permutations(list(range(cols)))))          # permuting columns permutes the result
    assert np.max(np.abs(oracle.softmax_rows(np.ascontiguousarray(Z[:, perm])) - P[:, perm])) <= 1e-13
    order = np.argsort(Z, axis=-1, kind="stable")                          # monotone in the scores
    sorted_p = np.take_along_axis(P, order, axis=-1)
    assert np.all(np.diff(sorted_p, axis=-1) >= -1e-15)


@settings(max_examples=40, deadline=None)
@given(st.integers(1, 3), st.integers(1, 12), st.sampled_from([8, 16]), st.integers(0, 2 ** 31 - 1),
       st.floats(min_value=0.0, max_value=2.0, allow_nan=False, width=32))
def test_attention_weight_invariants(heads, n, d, seed, scale):
    q = inputs.normal_bf16_bits(seed, 1, heads * n * d, 1.0).reshape(1, heads, n, d)
    k = inputs.normal_bf16_bits(seed, 2, heads * n * d, 1.0).reshape(1, heads, n, d)
    P = oracle.attnw(q, k, float(np.float32(scale)))
    assert P.shape == (1, heads, n, n) and np.all(P >= 0.0) and np.all(P <= 1.0)
    assert np.max(np.abs(P.sum(-1) - 1.0)) <= 1e-12
    same = np.broadcast_to(k[:, :, :1, :], k.shape).copy()                 # identical keys: exactly uniform
    assert np.array_equal(oracle.attnw(q, same, float(np.float32(scale))), np.full((1, heads, n, n), 1.0 / n))
    one = oracle.attnw(q[:, :1], k[:, :1], float(np.float32(scale)))       # heads are independent
    assert np.array_equal(one[0, 0], P[0, 0])


@settings(max_examples=200, deadline=None)
@given(st.integers(0, 5000), st.integers(1, 300))
def test_shard_range_partitions(total, world):
    cuts = [inputs.shard_range(total, r, world) for r in range(world)]
    assert cuts[0][0] == 0 and cuts[-1][1] == total
    assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
    sizes = [e - b for b, e in cuts]
    assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        inputs.shard_range(total, world, world)
