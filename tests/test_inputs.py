"""The seeded generator: reproducible, sliceable, and with the stated distribution."""
import numpy as np
import pytest

from paper_2407_13885_b200 import inputs


def test_reproducible_and_sliceable():
    a = inputs.normal_f32(inputs.SEED, 6, 10001, 2.0)
    b = inputs.normal_f32(inputs.SEED, 6, 10001, 2.0)
    assert np.array_equal(a, b)
    for off, cnt in [(0, 1), (1, 1), (3, 998), (4, 1000), (9999, 2), (10000, 1), (5, 0)]:
        assert np.array_equal(inputs.normal_f32(inputs.SEED, 6, cnt, 2.0, offset=off), a[off:off + cnt])


def test_streams_and_seeds_differ():
    a = inputs.normal_f32(1, 0, 1000, 1.0)
    assert not np.array_equal(a, inputs.normal_f32(1, 1, 1000, 1.0))
    assert not np.array_equal(a, inputs.normal_f32(2, 0, 1000, 1.0))


def test_moments():
    x = inputs.normal_f32(inputs.SEED, 3, 2_000_000, 3.0).astype(np.float64)
    assert abs(x.mean()) < 0.01
    assert abs(x.std() - 3.0) < 0.01
    assert abs(np.mean((x / 3.0) ** 4) - 3.0) < 0.05     # kurtosis of a normal
    assert abs(np.corrcoef(x[0::2], x[1::2])[0, 1]) < 0.005  # the two Box-Muller outputs


def test_bf16_round_to_nearest_even():
    f = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0],
                 dtype=np.float32)
    got = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(f))
    #            exact  tie->even(down)  tie->even(up)      above tie -> up             exact exact
    expect = np.array([1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -2.5, 0.0], dtype=np.float32)
    assert np.array_equal(got, expect)
    import torch
    x = inputs.normal_f32(5, 5, 100000, 4.0)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(inputs.f32_to_bf16_bits(x), ref)


def test_workloads_match_the_stated_configs():
    w = inputs.WORKLOADS
    assert (w["c1"].N, w["c1"].d, w["c1"].p_dtype, w["c1"].scale) == (256, 64, "f32", 0.125)
    assert (w["c2"].H, w["c2"].N, w["c2"].d) == (12, 2048, 64)
    assert (w["c3"].B, w["c3"].H, w["c3"].N, w["c3"].d) == (4, 32, 4096, 128)
    assert w["c3"].elements == 2 ** 31 and w["c3"].p_bytes == 2 ** 32
    assert (w["c4"].rows, w["c4"].cols, w["c4"].sigma) == (32768, 8192, 3.0)
    assert (w["c5"].H, w["c5"].N, w["c5"].sigma) == (8, 16384, 4.0)
    assert w["c3"].scale == float(np.float32(1 / np.sqrt(128.0)))


def test_make_qk_slices_agree():
    w = inputs.Workload("t", "fused", B=2, H=3, N=16, d=8, cfg_id=9)
    q, k = inputs.make_qk(w)
    q2, k2 = inputs.make_qk(w, 2, 5)
    assert q.shape == (6, 16, 8) and q.dtype == np.uint16
    assert np.array_equal(q[2:5], q2) and np.array_equal(k[2:5], k2)
    assert not np.array_equal(q, k)


@pytest.mark.parametrize("total,world", [(128, 8), (7, 4), (3, 8), (0, 2), (96, 5)])
def test_shard_range_covers_everything_once(total, world):
    spans = [inputs.shard_range(total, r, world) for r in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == total
    sizes = [e - b for b, e in spans]
    assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
