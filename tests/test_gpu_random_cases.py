"""Seeded random cases through the whole path against the oracle (needs a B200): layer sizes around the chunk and
sub-chunk boundaries, eight formats (flushed and not), 1 to 23 clients, strides with and without 16-byte alignment,
several decays, non-finite and huge inputs; two rounds each: memory, counters, streams, average, symbols, histogram."""
import numpy as np
import pytest

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, fmt_tuple, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits

pytestmark = pytest.mark.gpu

FORMATS = [(2, 1), (3, 0), (4, 3), (5, 2), (3, 2), (2, 3), (4, 1), (6, 1)]


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases(seed):
    rng = np.random.default_rng(seed)
    for _ in range(40):
        _one_case(rng)


def _one_case(rng):
    n_seg = int(rng.integers(1, 7))
    sizes = []
    for _ in range(n_seg):
        kind = rng.integers(0, 6)
        sizes.append(int([0, rng.integers(1, 40), rng.integers(2040, 2056), rng.integers(4090, 4104),
                          rng.integers(1, 30000), rng.integers(30000, 120000)][kind]))
    if sum(sizes) == 0:
        sizes[0] = 17
    fmts = []
    betas = []
    for k in range(n_seg):
        E, M = FORMATS[rng.integers(0, len(FORMATS))]
        beta = float(rng.uniform(0.6, 1.6))
        alpha = float(10 ** rng.uniform(-4, -1))
        betas.append((beta, alpha))
        tabulated = (E, M) in [(2, 1), (3, 0), (4, 3), (5, 2)]
        base = scale_for(E, M, beta, alpha)[0] if tabulated else 2.0 ** ((1 << (E - 1)) - 1) / (6 * alpha)
        sc = base * float(2 ** rng.uniform(-2, 2))
        fmts.append(fmt_tuple(E, M, sc, flush=bool(rng.integers(0, 4) == 0)))
    n_clients = int(rng.choice([1, 1, 2, 3, 5, 17, 23]))
    if n_clients > 5 and sum(sizes) > 60000:
        n_clients = 3
    stride = sum(sizes) + int(rng.choice([0, 0, 1, 3, 4, 13, 64]))
    decay = float(rng.choice([0.0, 0.5, 0.9, 1.0]))
    case = Case(sizes, fmts, n_clients=n_clients, decay=decay, stride=stride)
    gpu = Gpu(case)
    mem_o = np.zeros((n_clients, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    codes = None
    for rnd in range(2):
        g = np.zeros((n_clients, case.n_elem), dtype=np.float32)
        for u in range(n_clients):
            for k, n in enumerate(sizes):
                a = case.offsets[k]
                g[u, a:a + n] = gennorm(n, betas[k][0], betas[k][1], seed=int(rng.integers(0, 1 << 30))).numpy()
        # a few special values
        for _ in range(int(rng.integers(0, 4))):
            u = int(rng.integers(0, n_clients))
            i = int(rng.integers(0, case.n_elem))
            g[u, i] = rng.choice(np.array([np.inf, -np.inf, np.nan, 1e30, -1e30, 0.0, -0.0, 1e-45], dtype=np.float32))
        syms, ghats, nsat, nnf = oracle_convert(case, g, mem_o)
        if codes is None:
            codes = oracle_codes(case, oracle_hist(case, syms))
        want = oracle_encode(case, syms, codes)
        ok_all = all(st == oracle.OK for st, _ in want)
        out = gpu.encode(g, mem_g, codes)
        mem_g = out["mem"]
        assert out["status"] == co3.OK and out["guard_ok"], (sizes, fmts, n_clients)
        assert same_bits(mem_g, mem_o), ("mem", sizes, fmts, n_clients, stride, decay)
        assert np.array_equal(out["res"]["n_saturated"], nsat) and np.array_equal(out["res"]["n_nonfinite"], nnf)
        for u in range(n_clients):
            st, s = want[u]
            if st == oracle.OK:
                assert np.array_equal(out["streams"][u], s), ("stream", sizes, fmts, n_clients, stride, decay, u)
            else:
                assert out["res"][u]["status"] != co3.OK
        if ok_all:
            streams = [s for _, s in want]
            st, avg = oracle.decode_aggregate(streams, case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
            agg = gpu.decode_aggregate(out["streams"], codes)
            assert agg["res"][0]["status"] == co3.OK and same_bits(agg["avg"][:case.n_elem], avg), ("avg", sizes, n_clients)
            conv = gpu.convert(g, np.zeros_like(g)) if rnd == 0 and decay == 0.0 else None
            if conv is not None:
                assert np.array_equal(conv["sym"], syms) and np.array_equal(conv["hist"], oracle_hist(case, syms))
