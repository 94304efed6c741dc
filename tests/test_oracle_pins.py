"""Pins for the CPU oracle: checks against what the definition and the mathematics fix.

None of these re-types the oracle's own formula.  They use invariants of Softmax, closed
forms, brute force of the un-shifted definition in extended precision, float64 library
routines, and the worked values the paper prints (tests/golden/).
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2407_13885_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    """float array -> bf16 bit patterns (values must be exactly representable where exactness matters)."""
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def dec(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def rand_qk(B, H, N, d, sigma=1.0, stream=100):
    n = B * H * N * d
    q = inputs.normal_bf16_bits(7, stream, n, sigma).reshape(B, H, N, d)
    k = inputs.normal_bf16_bits(7, stream + 1, n, sigma).reshape(B, H, N, d)
    return q, k


# ---- invariants of the definition (Section VI) ------------------------------------------

@pytest.mark.parametrize("shape", [(1, 1, 4, 8), (2, 3, 37, 64), (1, 2, 256, 128)])
def test_rows_sum_to_one_and_range(shape):
    q, k = rand_qk(*shape)
    P = oracle.attnw(q, k, 1.0 / math.sqrt(shape[3]))
    assert P.shape == shape[:3] + (shape[2],)
    assert np.all(P >= 0.0) and np.all(P <= 1.0)
    assert np.max(np.abs(P.sum(-1) - 1.0)) <= 1e-12


@pytest.mark.parametrize("N", [1, 2, 3, 7, 64, 100, 1000, 4096])
def test_identical_keys_give_exactly_one_over_n(N):
    d = 16
    q = inputs.normal_bf16_bits(1, 5, N * d, 1.0).reshape(1, 1, N, d)
    one_key = inputs.normal_bf16_bits(1, 6, d, 1.0)
    k = np.tile(one_key, (N, 1)).reshape(1, 1, N, d)
    P = oracle.attnw(q, k, 0.25)
    assert np.array_equal(P, np.full_like(P, 1.0 / N))  # bit-exact


def test_zero_queries_or_zero_scale_give_uniform():
    q, k = rand_qk(1, 2, 33, 32)
    P = oracle.attnw(np.zeros_like(q), k, 0.3)
    assert np.array_equal(P, np.full_like(P, 1.0 / 33))
    P = oracle.attnw(q, k, 0.0)
    assert np.array_equal(P, np.full_like(P, 1.0 / 33))


def test_single_key_gives_one():
    q, k = rand_qk(2, 2, 1, 64)
    assert np.array_equal(oracle.attnw(q, k, 0.125), np.ones((2, 2, 1, 1)))


def test_permuting_keys_permutes_columns():
    q, k = rand_qk(1, 2, 129, 64)
    perm = np.random.default_rng(3).permutation(129)
    P = oracle.attnw(q, k, 0.125)
    Pp = oracle.attnw(q, k[:, :, perm, :], 0.125)
    assert np.max(np.abs(Pp - P[:, :, :, perm])) <= 1e-14


def test_heads_are_independent():
    q, k = rand_qk(2, 3, 40, 32)
    P = oracle.attnw(q, k, 0.2)
    for b in range(2):
        for h in range(3):
            Pbh = oracle.attnw(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], 0.2)
            assert np.array_equal(Pbh[0, 0], P[b, h])


def test_shift_invariance_eq1():
    """Adding 1*v^T to K adds the per-row constant q_i.v to every score of row i (Eq. 1)."""
    rng = np.random.default_rng(11)
    N, d = 24, 16
    qv = rng.integers(-3, 4, size=(1, 1, N, d)).astype(np.float32)
    kv = rng.integers(-3, 4, size=(1, 1, N, d)).astype(np.float32)
    v = rng.integers(-2, 3, size=(d,)).astype(np.float32)
    P0 = oracle.attnw(bits(qv), bits(kv), 0.125)
    P1 = oracle.attnw(bits(qv), bits(kv + v), 0.125)  # small integers: exact in bf16
    assert np.max(np.abs(P0 - P1)) <= 1e-15


def test_monotone_in_scores():
    S = inputs.normal_f32(5, 1, 6 * 50, 3.0).reshape(6, 50)
    P = oracle.softmax_rows(S)
    for i in range(6):
        order = np.argsort(S[i], kind="stable")
        assert np.all(np.diff(P[i][order]) >= 0.0)


# ---- closed forms -----------------------------------------------------------------------

def test_two_keys_logistic():
    for z1, z2 in [(0.0, 0.0), (1.5, -2.25), (-7.0, 3.0), (30.0, 29.5)]:
        S = np.array([[z1, z2]], dtype=np.float32)
        P = oracle.softmax_rows(S)
        expect = 1.0 / (1.0 + math.exp(-(z1 - z2)))
        assert abs(P[0, 0] - expect) <= 2e-16 * 4
        assert abs(P[0, 1] - (1.0 - expect)) <= 1e-15


def test_two_keys_logistic_through_attention():
    # d = 1: s_ij = q_i * k_j.  q = (1, 2), k = (0, 1): S = [[0, 1], [0, 2]] - not symmetric,
    # so swapping the operands (K Q^T) or transposing the result gives different rows.
    q = bits(np.array([1.0, 2.0]).reshape(1, 1, 2, 1))
    k = bits(np.array([0.0, 1.0]).reshape(1, 1, 2, 1))
    P = oracle.attnw(q, k, 0.5)
    e0 = 1.0 / (1.0 + math.exp(0.5))   # row 0: z = (0, 0.5)
    e1 = 1.0 / (1.0 + math.exp(1.0))   # row 1: z = (0, 1.0)
    expect = np.array([[e0, 1 - e0], [e1, 1 - e1]])
    assert np.max(np.abs(P[0, 0] - expect)) <= 1e-15


def test_arithmetic_progression_geometric_series():
    n, delta = 64, 0.25
    S = (np.arange(n) * delta).astype(np.float32).reshape(1, n)  # exact in fp32
    P = oracle.softmax_rows(S)
    r = math.exp(-delta)
    l = (1.0 - r ** n) / (1.0 - r)  # sum_{t=0}^{n-1} r^t, t = n-1-j
    expect = np.array([math.exp((j - (n - 1)) * delta) / l for j in range(n)])
    assert np.max(np.abs(P[0] - expect) / expect) <= 1e-13


def test_one_hot_limit_and_overflow_safety():
    S = np.zeros((2, 9), dtype=np.float32)
    S[0, 4] = 800.0            # exceeds the rest by more than 745: exp underflows to 0 in fp64
    S[1, :] = 1.0e4            # un-shifted exp would overflow; shifted row is uniform
    S[1, 2] = -1.0e4
    P = oracle.softmax_rows(S)
    expect0 = np.zeros(9)
    expect0[4] = 1.0
    assert np.array_equal(P[0], expect0)
    expect1 = np.full(9, 1.0 / 8)
    expect1[2] = 0.0
    assert np.array_equal(P[1], expect1)
    assert np.all(np.isfinite(P))


def test_large_logits_equal_shifted_row():
    base = inputs.normal_f32(9, 9, 128, 4.0).reshape(1, 128)
    big = (base.astype(np.float64) + 4096.0).astype(np.float32)  # shift by a power of two
    small = (big.astype(np.float64) - 4096.0).astype(np.float32)  # exact difference
    assert np.max(np.abs(oracle.softmax_rows(big) - oracle.softmax_rows(small))) <= 1e-15


def test_golden_log_integers():
    """tests/golden/softmax_log_integers.txt: Z_j = ln a_j gives a_j / sum a (Section VI)."""
    with open(os.path.join(GOLDEN, "softmax_log_integers.txt")) as f:
        rows = [list(map(int, ln.split())) for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 5
    for a in rows:
        a = np.array(a, dtype=np.float64)
        for shift in (0.0, 37.5, -120.0):
            S = (np.log(a) + shift).astype(np.float32).reshape(1, -1)
            P = oracle.softmax_rows(S)
            tol = 3e-7 * max(1.0, abs(shift))  # float32 rounding of the scores, nothing else
            assert np.max(np.abs(P[0] - a / a.sum())) <= tol


# ---- brute force of the un-shifted definition, extended precision ----------------------

def test_brute_force_4x4_long_double():
    rng = np.random.default_rng(2024)
    for trial in range(20):
        N, d = 4, 4
        qv = (rng.integers(-8, 9, size=(N, d)) / 4.0).astype(np.float32)  # exact in bf16
        kv = (rng.integers(-8, 9, size=(N, d)) / 4.0).astype(np.float32)
        scale = np.float32(0.5)
        P = oracle.attnw(bits(qv.reshape(1, 1, N, d)), bits(kv.reshape(1, 1, N, d)), float(scale))[0, 0]
        ld = np.longdouble
        for i in range(N):
            e = []
            for j in range(N):
                s = ld(0)
                for c in range(d):
                    s += ld(qv[i, c]) * ld(kv[j, c])
                e.append(np.exp(ld(scale) * s))       # no max subtraction: nothing overflows here
            tot = sum(e)
            for j in range(N):
                assert abs(float(e[j] / tot) - P[i, j]) <= 1e-13


def test_brute_force_rows_tiny():
    S = np.array([[0.5, -1.0, 2.0], [3.0, 3.0, -3.0]], dtype=np.float32)
    P = oracle.softmax_rows(S)
    for i in range(2):
        e = [math.exp(float(x)) for x in S[i]]
        for j in range(3):
            assert abs(P[i, j] - e[j] / sum(e)) <= 1e-15


# ---- float64 library routines on the same decoded inputs --------------------------------

@pytest.mark.parametrize("shape,sigma", [((1, 1, 256, 64), 1.0), ((2, 2, 200, 128), 4.0), ((1, 3, 77, 64), 1.0)])
def test_against_float64_library_softmax(shape, sigma):
    q, k = rand_qk(*shape, sigma=sigma, stream=300)
    scale = float(np.float32(1.0 / math.sqrt(shape[3])))
    P = oracle.attnw(q, k, scale)
    Z = scale * np.einsum("bhic,bhjc->bhij", dec(q), dec(k))
    ref = scipy.special.softmax(Z, axis=-1)
    assert np.max(np.abs(P - ref)) <= 1e-13
    ref_t = torch.softmax(torch.from_numpy(Z), dim=-1).numpy()
    assert np.max(np.abs(P - ref_t)) <= 1e-13


def test_rows_against_float64_library_softmax():
    S = inputs.normal_f32(3, 8, 33 * 1000, 3.0).reshape(33, 1000)
    P = oracle.softmax_rows(S)
    ref = scipy.special.softmax(S.astype(np.float64), axis=-1)
    assert np.max(np.abs(P - ref)) <= 1e-14
    sub = oracle.softmax_rows(S, rows_subset=[32, 0, 7])
    assert np.array_equal(sub, P[[32, 0, 7]])


def test_scores_step_alone():
    q, k = rand_qk(1, 2, 19, 64, stream=500)
    ids = np.array([0, 18, 19, 37])
    S = oracle.scores_rows(q, k, ids)
    full = np.einsum("bhic,bhjc->bhij", dec(q), dec(k)).reshape(2 * 19, 19)
    assert np.max(np.abs(S - full[ids])) <= 1e-12


def test_row_subset_matches_full():
    q, k = rand_qk(2, 2, 50, 64, stream=700)
    P = oracle.attnw(q, k, 0.125).reshape(-1, 50)
    ids = np.array([0, 49, 50, 123, 199])
    assert np.array_equal(oracle.attnw_rows(q, k, 0.125, ids), P[ids])


def test_scale_is_the_float32_value():
    """The oracle multiplies by the float32 scale widened to double, not by 1/sqrt(d) in double."""
    q, k = rand_qk(1, 1, 16, 128, sigma=4.0, stream=900)
    s32 = np.float32(1.0 / math.sqrt(128.0))
    P = oracle.attnw(q, k, float(s32))
    Z = float(s32) * np.einsum("bhic,bhjc->bhij", dec(q), dec(k))
    assert np.max(np.abs(P - scipy.special.softmax(Z, axis=-1))) <= 1e-13


def test_thread_count_does_not_change_results():
    q, k = rand_qk(1, 2, 65, 64, stream=40)
    assert np.array_equal(oracle.attnw(q, k, 0.125, threads=1), oracle.attnw(q, k, 0.125, threads=5))


# ---- the paper's own CPU program (Section VI-A), fp32 ----------------------------------

@pytest.mark.parametrize("variant", ["caching", "recomputing"])
def test_paper_cpu_program_agrees_with_oracle(variant):
    S = inputs.normal_f32(3, 77, 16 * 512, 3.0).reshape(16, 512)
    got = oracle.paper_cpu_softmax(S, variant).astype(np.float64)
    assert np.max(np.abs(got - oracle.softmax_rows(S))) <= 2e-6
    assert np.max(np.abs(got.sum(-1) - 1.0)) <= 1e-4


# ---- printed worked values of the row partition (Section VI-B) --------------------------

def test_row_partition_golden():
    with open(os.path.join(GOLDEN, "row_partition.txt")) as f:
        cases = [list(map(int, ln.split())) for ln in f if ln.strip() and not ln.startswith("#")]
    assert cases
    for units, workers, quotient, extra in cases:
        sizes = [e - b for b, e in (inputs.shard_range(units, r, workers) for r in range(workers))]
        assert sum(sizes) == units
        assert sizes[:extra] == [quotient + 1] * extra
        assert sizes[extra:] == [quotient] * (workers - extra)
        # contiguous, in order, starting from the first worker
        assert inputs.shard_range(units, 0, workers)[0] == 0
        for r in range(workers - 1):
            assert inputs.shard_range(units, r, workers)[1] == inputs.shard_range(units, r + 1, workers)[0]


# ---- the product with V: Attention(Q, K, V) of Section IV --------------------------------

def rand_v(B, H, N, d, sigma=1.0, stream=500):
    return inputs.normal_bf16_bits(7, stream, B * H * N * d, sigma).reshape(B, H, N, d)


def test_attention_of_constant_values_is_that_constant():
    q, k = rand_qk(1, 2, 50, 64, stream=510)
    v = bits(np.full((1, 2, 50, 64), 1.5, dtype=np.float32))
    O = oracle.attn(q, k, v, 0.125)
    assert np.max(np.abs(O - 1.5)) <= 1e-14          # rows of P sum to one


def test_attention_with_unit_vector_values_gives_column_sums_of_the_weights():
    N, d = 40, 8
    q, k = rand_qk(1, 1, N, d, stream=520)
    vv = np.zeros((1, 1, N, d), dtype=np.float32)
    for j in range(N):
        vv[0, 0, j, j % d] = 1.0
    O = oracle.attn(q, k, bits(vv), 0.3)[0, 0]
    P = oracle.attnw(q, k, 0.3)[0, 0]
    for c in range(d):
        assert np.max(np.abs(O[:, c] - P[:, c::d].sum(axis=1))) <= 1e-14


def test_attention_with_identical_keys_is_the_mean_value_and_single_key_is_its_value():
    N, d = 64, 16
    q, _ = rand_qk(1, 1, N, d, stream=530)
    key = inputs.normal_bf16_bits(5, 5, d, 1.0)
    kk = np.broadcast_to(key, (1, 1, N, d)).copy()
    vals = (np.arange(N * d).reshape(1, 1, N, d) % 17 - 8).astype(np.float32) / 4.0   # exact in bf16
    O = oracle.attn(q, kk, bits(vals), 0.7)[0, 0]
    assert np.max(np.abs(O - vals[0, 0].astype(np.float64).mean(axis=0))) <= 1e-13
    q1, k1 = rand_qk(1, 1, 1, d, stream=531)
    v1 = rand_v(1, 1, 1, d, stream=532)
    assert np.array_equal(oracle.attn(q1, k1, v1, 0.25)[0, 0, 0], dec(v1)[0, 0, 0])


def test_attention_is_linear_in_the_values():
    q, k = rand_qk(1, 1, 30, 32, stream=540)
    a = (np.random.default_rng(1).integers(-16, 17, size=(1, 1, 30, 32)) / 8.0).astype(np.float32)
    b = (np.random.default_rng(2).integers(-16, 17, size=(1, 1, 30, 32)) / 8.0).astype(np.float32)
    Oa, Ob = oracle.attn(q, k, bits(a), 0.2), oracle.attn(q, k, bits(b), 0.2)
    Oab = oracle.attn(q, k, bits(a + 2 * b), 0.2)     # a + 2b stays exact in bf16 (multiples of 1/8 below 8)
    assert np.max(np.abs(Oab - (Oa + 2 * Ob))) <= 1e-13


def test_attention_brute_force_4x4_long_double():
    rng = np.random.default_rng(77)
    ld = np.longdouble
    for trial in range(20):
        N, d = 4, 4
        qv = (rng.integers(-8, 9, size=(N, d)) / 4.0).astype(np.float32)
        kv = (rng.integers(-8, 9, size=(N, d)) / 4.0).astype(np.float32)
        vv = (rng.integers(-8, 9, size=(N, d)) / 4.0).astype(np.float32)
        scale = np.float32(0.5)
        O = oracle.attn(bits(qv.reshape(1, 1, N, d)), bits(kv.reshape(1, 1, N, d)), bits(vv.reshape(1, 1, N, d)),
                        float(scale))[0, 0]
        for i in range(N):
            e = [np.exp(ld(scale) * sum(ld(qv[i, c]) * ld(kv[j, c]) for c in range(d))) for j in range(N)]
            tot = sum(e)
            for c in range(d):
                want = sum(e[j] / tot * ld(vv[j, c]) for j in range(N))
                assert abs(float(want) - O[i, c]) <= 1e-13


@pytest.mark.parametrize("shape,sigma", [((1, 2, 100, 64), 1.0), ((2, 1, 77, 128), 4.0)])
def test_attention_against_float64_library(shape, sigma):
    q, k = rand_qk(*shape, sigma=sigma, stream=550)
    v = rand_v(*shape, stream=552)
    scale = float(np.float32(1.0 / math.sqrt(shape[3])))
    O = oracle.attn(q, k, v, scale)
    Z = scale * np.einsum("bhic,bhjc->bhij", dec(q), dec(k))
    ref = np.einsum("bhij,bhjc->bhic", scipy.special.softmax(Z, axis=-1), dec(v))
    assert np.max(np.abs(O - ref)) <= 1e-12
    ids = [0, 5, shape[0] * shape[1] * shape[2] - 1]
    assert np.array_equal(oracle.attn(q, k, v, scale, row_ids=ids), O.reshape(-1, shape[3])[ids])


# ---- queries and keys from the inputs: the linear transformation of Section IV ----------------

def rand_xw(B, N, d_model, H, d, sigma_w=None, stream=600):
    x = inputs.normal_bf16_bits(7, stream, B * N * d_model, 1.0).reshape(B, N, d_model)
    w = inputs.normal_bf16_bits(7, stream + 1, H * d * d_model, sigma_w or d_model ** -0.5).reshape(H, d, d_model)
    return x, w


def test_projection_with_selector_weights_copies_input_columns():
    # W[h, c, :] = unit vector e_{h*d + c}: head h of the output is columns h*d .. h*d+d-1 of X, exactly.
    B, N, H, d = 2, 9, 3, 4
    d_model = H * d + 5
    x, _ = rand_xw(B, N, d_model, H, d)
    w = np.zeros((H, d, d_model), dtype=np.float32)
    for h in range(H):
        for c in range(d):
            w[h, c, h * d + c] = 1.0
    out = oracle.project(x, bits(w))
    for h in range(H):
        assert np.array_equal(out[:, h], dec(x)[:, :, h * d:(h + 1) * d])   # catches swapped head / feature axes


def test_projection_small_integers_exact_and_brute_force():
    rng = np.random.default_rng(5)
    B, N, d_model, H, d = 2, 3, 6, 2, 3
    xv = rng.integers(-4, 5, size=(B, N, d_model)).astype(np.float32)
    wv = rng.integers(-4, 5, size=(H, d, d_model)).astype(np.float32)
    out = oracle.project(bits(xv), bits(wv))
    for b in range(B):
        for h in range(H):
            for n in range(N):
                for c in range(d):
                    want = sum(int(xv[b, n, m]) * int(wv[h, c, m]) for m in range(d_model))   # integers: exact
                    assert out[b, h, n, c] == want


def test_projection_is_linear_and_heads_are_independent():
    x, w = rand_xw(1, 20, 48, 2, 8, stream=610)
    out = oracle.project(x, w)
    w2 = dec(w).copy()
    w2[1] *= 2.0                                   # exact in bf16
    out2 = oracle.project(x, bits(w2.astype(np.float32)))
    assert np.array_equal(out2[:, 0], out[:, 0])
    assert np.array_equal(out2[:, 1], 2.0 * out[:, 1])
    x0 = dec(x).copy()
    x0[:, 7] = 0.0                                 # a zero input row gives a zero output row in every head
    assert np.all(oracle.project(bits(x0.astype(np.float32)), w)[:, :, 7] == 0.0)


def test_projection_against_float64_library_and_row_subset():
    B, N, d_model, H, d = 2, 33, 96, 3, 16
    x, w = rand_xw(B, N, d_model, H, d, stream=620)
    out = oracle.project(x, w)
    ref = np.einsum("bnm,hcm->bhnc", dec(x), dec(w))
    assert np.max(np.abs(out - ref)) <= 1e-13 * d_model
    ids = [0, 40, B * H * N - 1]
    assert np.array_equal(oracle.project(x, w, row_ids=ids), out.reshape(-1, d)[ids])
