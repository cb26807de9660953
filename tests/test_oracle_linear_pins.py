"""Pins of the linear / RMS-norm oracle against things other than itself: pure
Python loops on small integers (exact in bf16 and fp64), closed forms, and
structure a wrong index or a transposed operand would break."""
import math

import numpy as np
import pytest

from oracle import linear_oracle as lo


def bf16_bits(a) -> np.ndarray:
    """Round-to-nearest-even float -> bf16 bits (values used here are exactly representable)."""
    f = np.asarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def test_widen_is_exact_on_known_patterns():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x8000, 0x4049], dtype=np.uint16)
    assert lo.widen(bits).tolist() == [1.0, -1.0, 2.0, 0.5, 0.0, -0.0, 3.140625]


def test_linear_equals_python_loops_on_small_integers():
    rng = np.random.default_rng(0)
    M, N, K = 5, 7, 9                                     # all different: a transposed operand cannot pass
    x = rng.integers(-8, 9, size=(M, K))
    w = rng.integers(-8, 9, size=(N, K))
    want = [[sum(int(x[m, k]) * int(w[n, k]) for k in range(K)) for n in range(N)] for m in range(M)]
    got = lo.linear(bf16_bits(x), bf16_bits(w))
    assert got.shape == (M, N) and got.tolist() == want


def test_linear_one_hot_rows_select_weight_columns_and_ones_sum_rows():
    rng = np.random.default_rng(1)
    N, K = 6, 8
    w = rng.integers(-100, 100, size=(N, K)).astype(np.float64) / 4   # exactly representable in bf16
    eye = np.eye(K)
    assert np.array_equal(lo.linear(bf16_bits(eye), bf16_bits(w)), w.T)     # row k of x picks w[:, k]
    ones = np.ones((1, K))
    assert np.array_equal(lo.linear(bf16_bits(ones), bf16_bits(w))[0], w.sum(axis=1))


def test_linear_rows_are_independent():
    """The row-level contract's premise on the reference side: a row's result does not
    depend on the other rows of the batch."""
    rng = np.random.default_rng(2)
    x = bf16_bits(rng.standard_normal((6, 32)))
    w = bf16_bits(rng.standard_normal((10, 32)))
    full = lo.linear(x, w)
    for m in range(6):
        assert np.array_equal(lo.linear(x[m:m + 1], w)[0], full[m])


def test_rmsnorm_closed_forms():
    K = 16
    w = np.arange(1, K + 1) / 8.0
    # a constant row c: mean square c^2, y = w * c / sqrt(c^2 + eps)
    for cval, eps in ((2.0, 0.0), (-0.5, 1e-5), (3.0, 0.25)):
        y = lo.rmsnorm(bf16_bits(np.full((1, K), cval)), bf16_bits(w), eps)[0]
        assert np.allclose(y, w * cval / math.sqrt(cval * cval + eps), rtol=1e-15, atol=0)
    # a single non-zero entry v at position j: mean square v^2 / K, so y_j = sign(v) sqrt(K) w_j
    x = np.zeros((1, K))
    x[0, 5] = -4.0
    y = lo.rmsnorm(bf16_bits(x), bf16_bits(w), 0.0)[0]
    assert np.count_nonzero(y) == 1 and y[5] == pytest.approx(-math.sqrt(K) * w[5], rel=1e-15)
    # scale invariance without eps, and the zero row with eps
    rng = np.random.default_rng(3)
    xr = rng.integers(-16, 17, size=(3, K)).astype(np.float64)
    a = lo.rmsnorm(bf16_bits(xr), bf16_bits(w), 0.0)
    b = lo.rmsnorm(bf16_bits(4 * xr), bf16_bits(w), 0.0)
    assert np.allclose(a, b, rtol=1e-15, atol=0)
    assert np.array_equal(lo.rmsnorm(bf16_bits(np.zeros((1, K))), bf16_bits(w), 1e-6)[0], np.zeros(K))


def test_rmsnorm_equals_python_loops():
    rng = np.random.default_rng(4)
    M, K = 3, 12
    x = rng.integers(-8, 9, size=(M, K)).astype(np.float64) / 2
    w = rng.integers(-8, 9, size=K).astype(np.float64) / 4
    eps = 1e-3
    got = lo.rmsnorm(bf16_bits(x), bf16_bits(w), eps)
    for m in range(M):
        ms = sum(float(v) * float(v) for v in x[m]) / K
        for k in range(K):
            assert got[m, k] == pytest.approx(float(x[m, k]) / math.sqrt(ms + eps) * float(w[k]), rel=1e-14, abs=0)
