"""Pins for the oracle's Huffman construction (Sec. IV-A (ii)): no GPU.

Checked against what the mathematics fixes for an optimal prefix code: Kraft equality, the entropy
bounds H <= L < H + 1, brute-force optimality on a five-symbol alphabet, dyadic weights, the cost of
an independent heap-based construction, prefix-freeness and canonical order.
"""
import heapq
import itertools
import math

import numpy as np
import pytest

import oracle

FORMATS = [(2, 0), (2, 1), (3, 0), (4, 3), (5, 2)]


def _valid(fmt):
    return [s for s in range(256) if oracle.symbol_valid(fmt, s)]


def _build(weights, fmt):
    ln, bits = oracle.code_arrays(oracle.code_build(np.asarray(weights, dtype=np.uint64), fmt))
    return ln.astype(int), bits.astype(np.int64)


def _heap_cost(ws):
    h = list(ws)
    heapq.heapify(h)
    cost = 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        cost += a + b
        heapq.heappush(h, a + b)
    return cost


@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_kraft_entropy_and_cost(E, M, seed):
    fmt = oracle.make_fmt(E, M)
    valid = _valid(fmt)
    rng = np.random.default_rng(seed)
    w = np.zeros(256, dtype=np.uint64)
    w[valid] = (rng.pareto(1.2, size=len(valid)) * 50 + 1).astype(np.uint64)
    ln, bits = _build(w, fmt)
    assert all(ln[s] == 0 for s in range(256) if s not in valid)
    assert all(1 <= ln[s] <= oracle.MAX_CODE_LEN for s in valid)
    assert sum(1 << (16 - ln[s]) for s in valid) == 1 << 16                # complete code
    p = w[valid] / w[valid].sum()
    H = -(p * np.log2(p)).sum()
    Lbar = (p * ln[valid]).sum()
    assert H - 1e-12 <= Lbar < H + 1
    assert int((w[valid].astype(object) * ln[valid]).sum()) == _heap_cost([int(x) for x in w[valid]])
    # prefix-free, canonical
    words = {s: format(int(bits[s]), "0%db" % ln[s]) for s in valid}
    for a, b in itertools.permutations(valid, 2):
        assert not words[b].startswith(words[a])
    order = sorted(valid, key=lambda s: (ln[s], s))
    vals = [int(words[s].ljust(16, "0"), 2) for s in order]
    assert vals == sorted(vals) and len(set(vals)) == len(vals)
    assert int(bits[order[0]]) == 0


def test_brute_force_optimal_five_symbols():
    """[1,2,0] has five symbols (0, +-1, +-2): compare with every length assignment that satisfies Kraft."""
    fmt = oracle.make_fmt(2, 0)
    valid = _valid(fmt)
    assert len(valid) == 5
    rng = np.random.default_rng(4)
    for _ in range(60):
        w = np.zeros(256, dtype=np.uint64)
        w[valid] = rng.integers(1, 40, size=5).astype(np.uint64)
        ln, _ = _build(w, fmt)
        cost = sum(int(w[s]) * ln[s] for s in valid)
        best = min(sum(int(w[s]) * l for s, l in zip(valid, ls))
                   for ls in itertools.product(range(1, 5), repeat=5)
                   if sum(2.0 ** -l for l in ls) <= 1.0)
        assert cost == best


def test_dyadic_weights_give_log_lengths():
    fmt = oracle.make_fmt(2, 1)
    valid = _valid(fmt)                        # 11 symbols
    assert len(valid) == 11
    lens = [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 10]
    w = np.zeros(256, dtype=np.uint64)
    for s, l in zip(valid, lens):
        w[s] = 1 << (10 - l)
    ln, _ = _build(w, fmt)
    assert [ln[s] for s in valid] == lens


def test_zero_weights_still_get_codewords_and_limit_holds():
    fmt = oracle.make_fmt(5, 2)
    valid = _valid(fmt)
    w = np.zeros(256, dtype=np.uint64)
    ln, _ = _build(w, fmt)                      # all weights raised to 1
    assert sorted(set(ln[valid])) in ([7, 8], [8])
    # Fibonacci weights would need a depth of len(valid) - 1 without the limit
    a, b = 1, 1
    for s in valid[:60]:
        w[s] = a
        a, b = b, a + b
    ln, _ = _build(w, fmt)
    assert max(ln[valid]) <= oracle.MAX_CODE_LEN
    assert sum(1 << (16 - ln[s]) for s in valid) == 1 << 16
    heavy = valid[59]
    assert ln[heavy] <= 2


def test_weight_sum_overflow_rejected():
    fmt = oracle.make_fmt(4, 3)
    w = np.full(256, np.uint64(1) << np.uint64(62), dtype=np.uint64)
    with pytest.raises(ValueError):
        oracle.code_build(w, fmt)
