"""Dithered conversion (the stochastic rounding Sec. II-B (ii) allows for) through the C ABI against the oracle
(needs a B200): same draws on both sides, so symbols, memory, counters and streams must be identical."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, oracle_codes, oracle_encode, oracle_hist, same_bits

pytestmark = pytest.mark.gpu


def _oracle_round(case, seed, g, mems):
    """One round through the oracle with the library's draw stream; mems updated in place."""
    syms = np.zeros((case.n_clients, case.n_elem), dtype=np.uint8)
    ghats = np.zeros((case.n_clients, case.n_elem), dtype=np.float32)
    nsat = np.zeros(case.n_clients, dtype=np.uint64)
    nnf = np.zeros(case.n_clients, dtype=np.uint64)
    for u in range(case.n_clients):
        for k in range(case.n_seg):
            a, b = case.offsets[k], case.offsets[k + 1]
            m = mems[u, a:b].copy()
            draws = oracle.dither_draws(seed, u, k, 0, int(b - a))
            r = oracle.convert_dithered(g[u, a:b], m, case.decay, case.ofmt(k), draws)
            mems[u, a:b] = m
            syms[u, a:b] = r["sym"]
            ghats[u, a:b] = r["ghat"]
            nsat[u] += r["n_saturated"]
            nnf[u] += r["n_nonfinite"]
    return syms, ghats, nsat, nnf


def _case(n_clients, decay=0.9):
    sizes = [30000, 10, 4099, 64, 2048, 70001, 1, 5000]
    layout = [(4, 3, 0), (2, 1, 0), (5, 2, 0), (3, 0, 0), (4, 3, 1), (2, 1, 0), (4, 3, 0), (3, 0, 1)]   # (E, M, flags)
    fmts = [(E, M, fl) + scale_for(E, M, 0.9, 1e-3) for (E, M, fl) in layout]
    return Case(sizes, fmts, n_clients=n_clients, decay=decay, stride=sum(sizes) + 4)


@pytest.mark.parametrize("n_clients", [1, 3])
def test_convert_and_encode_with_dither_equal_the_oracle_over_rounds(n_clients):
    case = _case(n_clients)
    gpu = Gpu(case)
    mem_o = np.zeros((n_clients, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    codes = None
    for rnd, seed in enumerate((11, 0xffffffff, 0, 123456789)):
        g = np.stack([gennorm(case.n_elem, 0.9, 1e-3, seed=500 + 10 * rnd + u).numpy() for u in range(n_clients)])
        if rnd == 1:
            g[0, 5] = np.inf
            g[n_clients - 1, 30003] = np.nan
            g[0, 40000] = 7.0                                                 # far beyond the largest level
            g[0, 100:140] = (np.arange(40) * 1e-9).astype(np.float32)        # deep in the sub-normal range of the format
            g[0, 140:150] = np.float32(1e-41)                                 # fp32 sub-normals
        syms, ghats, nsat, nnf = _oracle_round(case, seed, g, mem_o)
        if rnd % 2 == 0:
            conv = gpu.convert(g, mem_g, dither_seed=seed)
            assert np.array_equal(conv["sym"], syms) and same_bits(conv["mem"], mem_o)
            assert np.array_equal(conv["hist"], oracle_hist(case, syms))
            assert np.array_equal(conv["res"]["n_saturated"], nsat) and np.array_equal(conv["res"]["n_nonfinite"], nnf)
            mem_g = conv["mem"]
        else:
            if codes is None:
                codes = oracle_codes(case, oracle_hist(case, syms))
            want = oracle_encode(case, syms, codes)
            out = gpu.encode(g, mem_g, codes, dither_seed=seed)
            assert same_bits(out["mem"], mem_o)
            assert np.array_equal(out["res"]["n_saturated"], nsat) and np.array_equal(out["res"]["n_nonfinite"], nnf)
            for u in range(n_clients):
                assert np.array_equal(out["streams"][u], want[u][1])
            dec = gpu.decode(out["streams"][0], codes)
            assert np.array_equal(dec["sym"][:case.n_elem], syms[0]) and same_bits(dec["ghat"][:case.n_elem], ghats[0])
            mem_g = out["mem"]


def test_draws_depend_on_seed_client_and_layer_only():
    """Two clients with the same gradient get different symbols; a second call with the same seed repeats the first;
    another seed changes the result; the dry histogram pass sees exactly what the round will produce."""
    n = 50000
    s, inv = scale_for(4, 3, 1.0, 1e-3)
    g1 = gennorm(n, 1.0, 1e-3, seed=9).numpy()
    g = np.stack([g1, g1])
    case = Case([n], [(4, 3, 0, s, inv)], n_clients=2, decay=0.0)
    outs = [Gpu(case).convert(g, np.zeros_like(g), dither_seed=seed) for seed in (1, 1, 2)]
    assert np.array_equal(outs[0]["sym"], outs[1]["sym"]) and same_bits(outs[0]["mem"], outs[1]["mem"])
    assert not np.array_equal(outs[0]["sym"], outs[2]["sym"])
    assert not np.array_equal(outs[0]["sym"][0], outs[0]["sym"][1])
    # unbiased: the mean error over many elements is statistically zero
    err = outs[0]["mem"].astype(np.float64)                     # m = v - ghat with zero old memory
    assert abs(err.mean()) < 4 * err.std() / np.sqrt(err.size)
    gpu = Gpu(case)
    hist = torch.zeros(256, dtype=torch.int64, device="cuda")
    gd, md = gpu._buf(g), gpu._buf(np.zeros_like(g))
    md0 = md.clone()
    assert co3.co3_histogram_dither(gd, md, 0.0, gpu.fmts, gpu.segs, 1, n, 2, case.stride, 1, hist, gpu.res, gpu.ws) == co3.OK
    torch.cuda.synchronize()
    assert np.array_equal(hist.cpu().numpy().astype(np.uint64), outs[0]["hist"][0]) and torch.equal(md, md0)


def test_many_chunks_and_clients():
    """Several chunks per block and layer, ten clients: the place of an element inside its layer drives the draws."""
    sizes = [300_000, 64, 700_001]
    fmts = [(4, 3, 0) + scale_for(4, 3, 1.0, 1e-3), (2, 1, 0) + scale_for(2, 1, 1.0, 1e-3), (5, 2, 0) + scale_for(5, 2, 1.0, 1e-3)]
    case = Case(sizes, fmts, n_clients=10, decay=0.7)
    g = np.stack([gennorm(case.n_elem, 1.0, 1e-3, seed=600 + u).numpy() for u in range(10)])
    m0 = np.stack([gennorm(case.n_elem, 2.0, 1e-4, seed=650 + u).numpy() for u in range(10)])
    mem_o = m0.copy()
    syms, _, nsat, _ = _oracle_round(case, 77, g, mem_o)
    conv = Gpu(case).convert(g, m0, dither_seed=77)
    assert np.array_equal(conv["sym"], syms) and same_bits(conv["mem"], mem_o)
    assert np.array_equal(conv["res"]["n_saturated"], nsat)
