"""Pins of the oracle's parameter-server model update (Algorithm 1, last step): w <- w - eta * avg."""
from fractions import Fraction

import numpy as np

import oracle


def _exact_step(w, avg, eta):
    """The result by exact rational arithmetic with the two roundings written out: fl(w - fl(eta * avg)).
    A product of two fp32 numbers has at most 48 significant bits, so it is exact in fp64 and np.float32()
    rounds it once; the inputs below keep |w| and |step| within 2^20 of each other, so their difference is
    exact in fp64 as well and is rounded once too."""
    out = np.empty_like(w)
    for i in range(w.size):
        prod = Fraction(float(eta)) * Fraction(float(avg[i]))
        step = np.float32(float(prod))
        assert Fraction(float(prod)) == prod
        diff = Fraction(float(w[i])) - Fraction(float(step))
        assert Fraction(float(diff)) == diff
        out[i] = np.float32(float(diff))
    return out


def test_update_matches_exact_arithmetic_rounded_twice():
    rng = np.random.default_rng(3)
    w = rng.standard_normal(4000).astype(np.float32)
    avg = (rng.standard_normal(4000) * 0.37).astype(np.float32)
    for eta in (np.float32(0.01), np.float32(0.3), np.float32(1.7)):
        got = w.copy()
        oracle.ps_update(got, avg, float(eta))
        want = _exact_step(w, avg, eta)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_zero_rate_and_zero_gradient_leave_the_model_alone():
    rng = np.random.default_rng(4)
    w = rng.standard_normal(1000).astype(np.float32)
    got = w.copy()
    oracle.ps_update(got, rng.standard_normal(1000).astype(np.float32), 0.0)
    assert np.array_equal(got.view(np.uint32), w.view(np.uint32))
    got = w.copy()
    oracle.ps_update(got, np.zeros(1000, dtype=np.float32), 0.25)
    assert np.array_equal(got.view(np.uint32), w.view(np.uint32))


def test_power_of_two_rate_from_zero_model_is_an_exact_scaling():
    rng = np.random.default_rng(5)
    avg = rng.standard_normal(1000).astype(np.float32)
    w = np.zeros(1000, dtype=np.float32)
    oracle.ps_update(w, avg, 0.125)
    assert np.array_equal(w, -avg / np.float32(8.0))          # exact in fp32: a change of exponent only
    assert (np.signbit(w) != np.signbit(avg))[avg != 0].all()  # the step goes against the gradient


def test_constant_gradient_walks_a_line():
    # T steps against a gradient whose products and partial sums are all exactly representable:
    # the model after T steps is w0 - T * eta * avg with no rounding at all (SGD recursion of Sec. II-A)
    w0 = np.arange(64, dtype=np.float32)
    avg = np.full(64, 3.0, dtype=np.float32)
    w = w0.copy()
    for _ in range(10):
        oracle.ps_update(w, avg, 0.5)
    assert np.array_equal(w, w0 - np.float32(15.0))
