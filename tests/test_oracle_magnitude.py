"""Pins of the oracle's error-magnitude figures (Sec. VI, "Error magnitude": l1 norm of the memory term
against the l1 norm of the gradient term)."""
import math
from fractions import Fraction

import numpy as np

import oracle
from co3_inputs import gennorm


def test_closed_forms():
    # constant magnitudes with mixed signs, and an arithmetic progression: n*a and n(n+1)/2 * step, exactly
    g = np.full(1000, -0.375, dtype=np.float32)
    g[::3] = 0.375
    m = (np.arange(1, 1001, dtype=np.float32) * np.float32(0.5)) * np.where(np.arange(1000) % 2, -1, 1).astype(np.float32)
    out = oracle.error_magnitude(g, m)
    assert out[0] == 375.0 and out[1] == 0.5 * 1000 * 1001 / 2
    assert np.array_equal(oracle.error_magnitude(np.zeros(0, np.float32), np.zeros(0, np.float32)), [0.0, 0.0])
    assert np.array_equal(oracle.error_magnitude(np.float32([-0.0, 0.0]), np.float32([2.0, -2.0])), [0.0, 4.0])


def test_against_exact_rational_sums_and_numpy():
    g = gennorm(20000, 0.8, 1e-3, 3).numpy()
    m = gennorm(20000, 1.2, 3e-4, 4).numpy()
    out = oracle.error_magnitude(g, m)
    for x, got in ((g, out[0]), (m, out[1])):
        exact = sum((Fraction(float(abs(v))) for v in x), Fraction(0))
        assert abs(Fraction(got) - exact) <= exact * Fraction(1, 10 ** 13)
        assert abs(got - np.abs(x.astype(np.float64)).sum()) <= 1e-12 * got
    # the two norms are not swapped, and scaling one input scales only its norm
    out2 = oracle.error_magnitude(g, np.float32(4.0) * m)
    assert out2[0] == out[0] and abs(out2[1] - 4.0 * out[1]) <= 1e-12 * out2[1]


def test_expected_size_for_the_model_and_nonfinite_inputs():
    # E|X| of GenNorm(0, alpha, beta) is alpha * Gamma(2/beta) / Gamma(1/beta)
    for beta, alpha in ((1.0, 2e-3), (2.0, 1e-2), (0.7, 5e-4)):
        x = gennorm(1 << 20, beta, alpha, 11).numpy()
        mean_abs = oracle.error_magnitude(x, x)[0] / x.size
        want = alpha * math.gamma(2.0 / beta) / math.gamma(1.0 / beta)
        assert abs(mean_abs - want) < 0.01 * want
    x = np.ones(10, dtype=np.float32)
    y = x.copy(); y[3] = np.nan
    out = oracle.error_magnitude(x, y)
    assert out[0] == 10.0 and math.isnan(out[1])
    y[3] = -np.inf
    assert oracle.error_magnitude(y, x)[0] == np.inf
