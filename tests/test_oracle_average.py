"""Pins of the checker's group mean (Algorithm 1: A <- allReduce(A / worldSize), same for B).
CPU only."""
import numpy as np
import pytest

from oracle import ab_oracle as orc
from paper_2405_01067_b200 import synth


def _copies(K, shape, seed=0, bf16=False):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal((K,) + shape).astype(np.float32)
    return synth.bf16_round(c) if bf16 else c


@pytest.mark.parametrize("K", [1, 2, 3, 4, 8])
def test_identical_copies_come_back_bit_for_bit(K):
    base = _copies(1, (37, 5))[0]
    c = np.stack([base] * K)
    out = orc.group_average_f32(c)
    if K in (1, 2):
        assert np.array_equal(out.view(np.uint32), base.view(np.uint32))
    else:
        # the running sum 3x, 5x, ... is rounded: within one rounding per step
        assert np.allclose(out, base, rtol=K * 2.0 ** -24, atol=0)
    assert np.allclose(orc.group_average(c), base.astype(np.float64), rtol=1e-15)


def test_two_copies_is_the_rounded_half_sum():
    c = _copies(2, (1000,), 1)
    expect = ((c[0].astype(np.float64) + c[1].astype(np.float64)) / 2).astype(np.float32)
    assert np.array_equal(orc.group_average_f32(c), expect)


@pytest.mark.parametrize("K", [2, 4, 8])
def test_prescaled_equals_postscaled_for_power_of_two(K):
    c = _copies(K, (4096,), K)
    a = orc.group_average_f32(c)
    b = orc.group_average_prescaled_f32(c)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


@pytest.mark.parametrize("K,bf16", [(3, False), (8, False), (4, True), (5, True)])
def test_fp32_mean_is_close_to_the_exact_mean(K, bf16):
    c = _copies(K, (513, 7), 10 + K, bf16)
    exact = orc.group_average(c)
    got = orc.group_average_f32(c).astype(np.float64)
    bound = K * 2.0 ** -24 * np.mean(np.abs(c.astype(np.float64)), axis=0) * K + 1e-30
    assert np.all(np.abs(got - exact) <= bound + 2.0 ** -24 * np.abs(exact))


def test_order_is_k_ascending():
    # (1 + 2^-24) + 2^-24 rounds differently from 1 + (2^-24 + 2^-24)
    c = np.array([[1.0], [2.0 ** -24], [2.0 ** -24], [0.0]], dtype=np.float32)
    out = orc.group_average_f32(c)
    assert out[0] == np.float32(0.25)              # both small addends are lost one after the other
    rev = orc.group_average_f32(c[::-1].copy())
    assert rev[0] == np.float32((1.0 + 2.0 ** -23) / 4)


def test_recombine_is_the_plain_product():
    rng = np.random.default_rng(4)
    A = rng.standard_normal((5, 3))
    B = rng.standard_normal((3, 4))
    W = orc.recombine(A, B)
    for i in range(5):
        for j in range(4):
            assert abs(W[i, j] - sum(A[i, k] * B[k, j] for k in range(3))) < 1e-14


def test_bf16_round_helper():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.3895313892515355e38, 0.1], dtype=np.float32)
    r = synth.bf16_round(x)
    assert r[0] == 1.0
    assert r[1] == 1.0                 # tie: 1 + 2^-8 rounds to even (1.0)
    assert r[2] == np.float32(1.015625)  # tie: 1 + 3*2^-8 rounds to even (1 + 2^-6)
    assert np.array_equal(synth.from_bf16_bits(synth.to_bf16_bits(r)), r)
    assert abs(r[4] - 0.1) < 0.1 * 2.0 ** -8
