"""Pins of the oracle's dithered converter (Sec. II-B (ii): the quantizer may be a stochastic mapping, for
non-subtractive dither).  The generator against its published test vectors; the rounding rule against what the
mathematics fixes: with every draw enumerated the mean of the result is the input itself, levels never move,
the result is always one of the two levels around the input, saturation and the memory recursion are unchanged."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "philox4x32_kat.txt")
N_DRAWS = 1 << 24


def _fmt(E, M, scale=1.0, flush=False):
    s = np.float32(scale)
    return oracle.Fmt(E, M, 1 if flush else 0, float(s), float(np.float32(1.0) / s))


def test_generator_reproduces_the_published_vectors():
    rows, nth = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("10000th"):
            nth = int(line.split()[1])
            continue
        c, k, o = [[int(x, 16) for x in part.split()] for part in line.split("|")]
        rows.append((c, k, o))
    assert len(rows) == 3 and nth is not None
    for c, k, o in rows:
        assert oracle.philox4x32_10(c, k).tolist() == o
    # the standard's engine: block b of the default-seeded stream is the function at counter (b, 0, 0, 0)
    i = 10000 - 1
    assert int(oracle.philox4x32_10([i // 4, 0, 0, 0], [20111115, 0])[i % 4]) == nth


def test_draws_follow_the_documented_counter_layout():
    d = oracle.dither_draws(seed=123, client=5, layer=9, first_place=6, n=7)      # places 6 .. 12
    for i, p in enumerate(range(6, 13)):
        block = oracle.philox4x32_10([p // 4, 0, 5, 9], [123, 0])
        assert d[i] == block[p % 4] >> 8
    far = oracle.dither_draws(1, 0, 0, (1 << 34) + 1, 1)                          # the place's high word
    assert far[0] == oracle.philox4x32_10([0, 1, 0, 0], [1, 0])[1] >> 8
    big = oracle.dither_draws(99, 3, 1, 0, 1 << 16)
    assert big.max() < N_DRAWS and abs(big.mean() / N_DRAWS - 0.5) < 0.01
    assert not np.array_equal(big, oracle.dither_draws(100, 3, 1, 0, 1 << 16))


def _all_draws(x, fmt):
    """Results for one input under every possible draw: (values, symbols)."""
    draws = np.arange(N_DRAWS, dtype=np.uint32)
    g = np.full(N_DRAWS, x, dtype=np.float32)
    r = oracle.convert_dithered(g, np.zeros(N_DRAWS, dtype=np.float32), 0.0, fmt, draws)
    return r["ghat"], r["sym"]


@pytest.mark.parametrize("E,M,flush", [(4, 3, False), (2, 1, False), (5, 2, False), (3, 0, False), (4, 3, True)])
def test_mean_over_all_draws_is_the_input(E, M, flush):
    """Exact rational arithmetic: sum of the 2^24 results = 2^24 * x for inputs from the smallest normal level up
    (and for sub-normal inputs on the 2^-24 grid of the step); the results are the two levels around x only."""
    fmt = _fmt(E, M, 1.0, flush)
    codes, lv = oracle.levels(fmt)
    emin = -((1 << (E - 1)) - 2)
    rng = np.random.default_rng(E * 10 + M)
    xs = [np.float32(2.0 ** emin * 1.3), np.float32(-(2.0 ** emin) * 1.999), np.float32(lv[-1] * 0.77),
          np.float32(rng.uniform(2.0 ** emin, lv[-1])), np.float32(2.0 ** emin * (1 + 2.0 ** -23))]
    xs.append(np.float32(2.0 ** emin * 0.37109375))                 # below the smallest normal level, on a coarse grid
    for x in xs:
        vals, syms = _all_draws(x, fmt)
        uniq, counts = np.unique(vals, return_counts=True)
        a = abs(float(x))
        below, above = lv[lv <= a].max(), lv[lv >= a].min()
        assert set(np.abs(uniq).tolist()) <= {below, above}
        total = sum(Fraction(float(u)) * int(c) for u, c in zip(uniq, counts))
        assert total == Fraction(float(x)) * N_DRAWS, (E, M, flush, x)


def test_probability_is_the_position_between_the_levels_rounded_up_to_the_draw_grid():
    """A sub-normal input off the 2^-24 grid: the number of draws that go up is ceil(position * 2^24)."""
    fmt = _fmt(4, 3)
    step = 2.0 ** (-6 - 3)
    x = np.float32(step * (2 + 1.0 / 3.0))                          # between levels 2 and 3 of the sub-normal run
    vals, _ = _all_draws(x, fmt)
    where = Fraction(float(x)) / Fraction(step) - 2
    want_up = -((-where * N_DRAWS) // 1)                            # ceiling
    assert int((vals == np.float32(3 * step)).sum()) == want_up
    assert abs(Fraction(float(vals.astype(np.float64).sum())) / N_DRAWS - Fraction(float(x))) < Fraction(step) / N_DRAWS


def test_levels_saturation_and_special_values_do_not_depend_on_the_draw():
    fmt = _fmt(4, 3, 3.0)
    codes, lv = oracle.levels(fmt)
    rng = np.random.default_rng(5)
    g = np.concatenate([lv, -lv[1:]]).astype(np.float32) / np.float32(3.0)
    g = g[(g * np.float32(3.0)).astype(np.float64).__abs__() == np.concatenate([lv, lv[1:]])]   # exact after scaling
    base = oracle.convert(g, np.zeros_like(g), 0.0, fmt)
    for _ in range(4):
        d = rng.integers(0, N_DRAWS, size=g.size, dtype=np.uint32)
        r = oracle.convert_dithered(g, np.zeros_like(g), 0.0, fmt, d)
        assert np.array_equal(r["sym"], base["sym"]) and np.array_equal(r["ghat"], base["ghat"])
    special = np.array([1e9, -1e9, np.inf, -np.inf, np.nan, 0.0, -0.0, 81.0, -80.0001], dtype=np.float32)
    want = oracle.convert(special, np.zeros_like(special), 0.0, fmt)
    for draw in (0, 1, N_DRAWS - 1):
        m = np.zeros_like(special)
        r = oracle.convert_dithered(special, m, 0.0, fmt, np.full(special.size, draw, dtype=np.uint32))
        assert np.array_equal(r["sym"], want["sym"]) and r["n_saturated"] == want["n_saturated"] == 4
        assert r["n_nonfinite"] == 3
    with pytest.raises(ValueError):
        oracle.convert_dithered(special, np.zeros_like(special), 0.0, fmt, np.full(special.size, N_DRAWS, dtype=np.uint32))


def test_extreme_draws_give_floor_and_ceiling_and_memory_recursion_holds():
    fmt = _fmt(5, 2, 100.0)
    rng = np.random.default_rng(11)
    g = (rng.standard_normal(20000) * 0.05).astype(np.float32)
    m0 = (rng.standard_normal(20000) * 0.01).astype(np.float32)
    codes, lv = oracle.levels(fmt)
    lo = oracle.convert_dithered(g, m0.copy(), 0.9, fmt, np.full(g.size, N_DRAWS - 1, dtype=np.uint32))
    hi = oracle.convert_dithered(g, m0.copy(), 0.9, fmt, np.zeros(g.size, dtype=np.uint32))
    v = (np.float32(0.9) * m0.astype(np.float64) + g.astype(np.float64)).astype(np.float32)      # one rounding: as fmaf
    t = np.abs((v * np.float32(100.0)).astype(np.float64))
    idx = np.searchsorted(lv, t, side="right") - 1
    floor_lv = lv[idx]
    ceil_lv = np.where(lv[idx] == t, t, lv[np.minimum(idx + 1, lv.size - 1)])
    inv = np.float32(fmt.inv_scale)
    assert np.array_equal(np.abs(lo["ghat"]), (floor_lv.astype(np.float32) * inv))
    assert np.array_equal(np.abs(hi["ghat"]), (ceil_lv.astype(np.float32) * inv))
    m = m0.copy()
    d = rng.integers(0, N_DRAWS, size=g.size, dtype=np.uint32)
    r = oracle.convert_dithered(g, m, 0.9, fmt, d)
    assert np.array_equal(m, v - r["ghat"])                          # m_t = (g + gamma m) - ghat, term by term
    # unbiased in the statistical sense too: the mean error over many elements is far below one step
    assert abs(float((r["ghat"].astype(np.float64) - v).mean())) < 3 * 0.05 * 2.0 ** -2 / np.sqrt(g.size)
