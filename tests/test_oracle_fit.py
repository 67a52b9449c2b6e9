"""Pins of the oracle's per-layer fit of the converter's multiplier (Sec. III: zero-mean GenNorm model with
its kurtosis and variance formulas; Sec. IV-A (i): the multiplier that minimises the conversion error)."""
import math

import numpy as np

import oracle
from co3_inputs import gennorm, scale_for

BETA0, DBETA, NB = 0.3, 0.05, 35
# the table's grid as the oracle sees it: both numbers are passed as fp32
GRID = float(np.float32(BETA0)) + float(np.float32(DBETA)) * np.arange(NB)


def _flat_table(c):
    return np.full(NB, math.log(c), dtype=np.float32)


def test_kurtosis_closed_forms():
    # Gamma at integers and half-integers: normal 3, Laplace 6, shape 1/2: Gamma(10) Gamma(2) / Gamma(6)^2
    assert abs(oracle.gennorm_kurtosis(2.0) - 3.0) < 1e-12
    assert abs(oracle.gennorm_kurtosis(1.0) - 6.0) < 1e-12
    assert abs(oracle.gennorm_kurtosis(0.5) - 362880.0 / 14400.0) < 1e-10
    ks = [oracle.gennorm_kurtosis(b) for b in np.linspace(0.3, 2.0, 50)]
    assert all(a > b for a, b in zip(ks, ks[1:]))     # heavier tails for smaller shapes


def test_shape_from_kurtosis_inverts_and_clamps():
    for b in (0.3, 0.45, 0.8, 1.0, 1.37, 1.99, 2.0):
        got = oracle.gennorm_shape_from_kurtosis(oracle.gennorm_kurtosis(b), 0.3, 2.0)
        assert abs(got - b) < 1e-9
    assert oracle.gennorm_shape_from_kurtosis(1.0, 0.3, 2.0) == 2.0       # lighter tails than a normal
    assert oracle.gennorm_shape_from_kurtosis(1e9, 0.3, 2.0) == 0.3


def test_two_point_and_three_point_layers_have_closed_forms():
    a, c = 0.25, 3.0
    # +-a only: sigma = a, kurtosis 1 -> shape clamped to 2 (normal): alpha = sigma * sqrt(2)
    g = np.tile(np.array([a, -a], dtype=np.float32), 500)
    st, sc, inv, stats = oracle.fit_scale(g, None, 0.0, _flat_table(c), BETA0, DBETA)
    assert st == oracle.OK
    assert abs(stats[0] - a) < 1e-15 and abs(stats[1] - 1.0) < 1e-15 and stats[2] == GRID[-1]
    assert abs(stats[3] - a * math.sqrt(math.gamma(1.0 / GRID[-1]) / math.gamma(3.0 / GRID[-1]))) < 1e-12
    assert abs(stats[3] - a * math.sqrt(2.0)) < 1e-7      # the grid's last node is 2 up to fp32 rounding
    assert sc == np.float32(c / stats[3]) and inv == np.float32(1.0) / np.float32(sc)
    # five zeros for every +-a: kurtosis exactly 6 -> Laplace: alpha = sigma / sqrt(2), sigma = a / sqrt(6)
    g = np.tile(np.array([a, 0, 0, 0, 0, 0, -a, 0, 0, 0, 0, 0], dtype=np.float32), 300)
    st, sc, inv, stats = oracle.fit_scale(g, None, 0.0, _flat_table(c), BETA0, DBETA)
    assert st == oracle.OK and abs(stats[1] - 6.0) < 1e-12 and abs(stats[2] - 1.0) < 1e-9
    assert abs(stats[3] - a / math.sqrt(12.0)) < 1e-10
    assert abs(sc - c * math.sqrt(12.0) / a) < 1e-4 * sc


def test_table_is_interpolated_linearly_in_the_logarithm():
    a = 0.25
    g = np.tile(np.array([a, 0, 0, 0, 0, 0, -a, 0, 0, 0, 0, 0], dtype=np.float32), 300)   # shape 1, alpha a/sqrt(12)
    alpha = a / math.sqrt(12.0)
    betas = GRID
    lin = (0.7 - 1.3 * betas).astype(np.float32)                     # exactly linear: any interpolation point is exact
    st, sc, _, _ = oracle.fit_scale(g, None, 0.0, lin, BETA0, DBETA)
    assert st == oracle.OK and abs(sc - math.exp(0.7 - 1.3) / alpha) < 2e-6 * sc
    # a layer whose kurtosis falls between two nodes: against numpy's interpolation of the same table
    rng = np.random.default_rng(0)
    tab = rng.standard_normal(NB).astype(np.float32)
    x = gennorm(400_000, 0.83, 1e-3, 77, "cpu").numpy()
    st, sc, _, stats = oracle.fit_scale(x, None, 0.0, tab, BETA0, DBETA)
    want = math.exp(float(np.interp(stats[2], betas, tab.astype(np.float64)))) / stats[3]
    assert st == oracle.OK and abs(sc - want) < 1e-7 * want
    assert betas[0] < stats[2] < betas[-1] and (stats[2] - BETA0) / DBETA % 1.0 > 1e-3


def test_moments_against_numpy_and_memory_correction():
    x = gennorm(300_000, 1.2, 2e-3, 5, "cpu").numpy().reshape(3, 100_000)      # three clients of one layer
    st, sc, _, stats = oracle.fit_scale(x, None, 0.0, _flat_table(1.0), BETA0, DBETA)
    x64 = x.astype(np.float64)
    assert st == oracle.OK
    assert abs(stats[0] - math.sqrt(np.mean(x64 ** 2))) < 1e-12 * stats[0]
    assert abs(stats[1] - np.mean(x64 ** 4) / np.mean(x64 ** 2) ** 2) < 1e-10 * stats[1]
    # v = g + decay * m: the fit of (g, m) is the fit of v formed first (decay 0.5: the product is exact)
    m = gennorm(300_000, 1.0, 1e-3, 6, "cpu").numpy().reshape(3, 100_000)
    v = (x.astype(np.float64) + 0.5 * m.astype(np.float64)).astype(np.float32)
    a = oracle.fit_scale(x, m, 0.5, _flat_table(1.0), BETA0, DBETA)
    b = oracle.fit_scale(v, None, 0.0, _flat_table(1.0), BETA0, DBETA)
    assert a[0] == b[0] == oracle.OK and a[1] == b[1] and np.array_equal(a[3], b[3])


def test_fit_recovers_the_generating_parameters():
    import json, os
    import co3_inputs
    with open(os.path.join(os.path.dirname(co3_inputs.__file__), "scale_table.json")) as fh:
        table = json.load(fh)
    for (E, M), beta, alpha in (((4, 3), 1.0, 1e-3), ((2, 1), 0.7, 3e-4), ((5, 2), 1.5, 1e-2)):
        tab = np.log(np.asarray(table["formats"]["%d,%d" % (E, M)], dtype=np.float64)).astype(np.float32)
        x = gennorm(2_000_000, beta, alpha, 123, "cpu").numpy()
        st, sc, inv, stats = oracle.fit_scale(x, None, 0.0, tab, BETA0, DBETA)
        assert st == oracle.OK
        assert abs(stats[2] - beta) < 0.05 * beta and abs(stats[3] - alpha) < 0.05 * alpha
        assert abs(sc - scale_for(E, M, beta, alpha)[0]) < 0.08 * sc      # the multiplier a known model would get


def test_layers_without_a_fit():
    tab = _flat_table(1.0)
    assert oracle.fit_scale(np.zeros(100, dtype=np.float32), None, 0.0, tab, BETA0, DBETA)[0] != oracle.OK
    x = np.ones(100, dtype=np.float32); x[7] = np.nan
    assert oracle.fit_scale(x, None, 0.0, tab, BETA0, DBETA)[0] != oracle.OK
    x[7] = np.inf
    assert oracle.fit_scale(x, None, 0.0, tab, BETA0, DBETA)[0] != oracle.OK
