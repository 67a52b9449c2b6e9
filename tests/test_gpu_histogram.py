"""co3_histogram (symbol statistics of this round without touching the memory) against the oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, fmt_tuple, oracle_convert, oracle_hist

pytestmark = pytest.mark.gpu


def _dry(case, gpu, g_np, m_np):
    c = case
    g, m = gpu._buf(g_np), gpu._buf(m_np)
    g0, m0 = g.clone(), m.clone()
    hist = torch.full((max(1, c.n_seg) * 256,), 9, dtype=torch.int64, device="cuda")
    st = co3.co3_histogram(g, m, c.decay, gpu.fmts, gpu.segs, c.n_seg, c.n_elem, c.n_clients, c.stride, hist, gpu.res,
                           gpu.ws)
    torch.cuda.synchronize()
    assert st == co3.OK
    assert torch.equal(g.view(torch.int32), g0.view(torch.int32)) and torch.equal(m.view(torch.int32), m0.view(torch.int32))
    return hist.cpu().numpy().astype(np.uint64).reshape(-1, 256)[:c.n_seg], co3.read_results(gpu.res, c.n_clients)


@pytest.mark.parametrize("n_clients", [1, 3])
def test_counts_equal_the_oracle_and_nothing_else_is_written(n_clients):
    sizes = [5000, 10, 64, 0, 2048, 4099, 1, 300000, 2047]
    fmts = []
    for k in range(len(sizes)):
        E, M = [(4, 3), (2, 1), (5, 2), (3, 0)][k % 4]
        fmts.append((E, M, k % 3 == 2) + scale_for(E, M, 0.9, 1e-3))
    fmts = [(E, M, 1 if fl else 0, s, inv) for (E, M, fl, s, inv) in fmts]
    case = Case(sizes, fmts, n_clients=n_clients, decay=0.9, stride=sum(sizes) + 4)
    g = np.stack([gennorm(case.n_elem, 0.9, 1e-3, seed=300 + u).numpy() for u in range(n_clients)])
    m = np.stack([gennorm(case.n_elem, 1.5, 2e-4, seed=350 + u).numpy() for u in range(n_clients)])
    g[0, 7] = np.inf
    g[n_clients - 1, 5100] = np.nan
    g[0, 20000] = 50.0                                          # far beyond the largest level
    gpu = Gpu(case)
    hist, res = _dry(case, gpu, g, m)
    mem_o = m.copy()
    syms, _, nsat, nnf = oracle_convert(case, g, mem_o)
    assert np.array_equal(hist, oracle_hist(case, syms))
    assert int(hist.sum()) == case.n_elem * n_clients
    assert np.array_equal(res["n_saturated"], nsat) and np.array_equal(res["n_nonfinite"], nnf)
    # the round itself, afterwards, sees the same statistics and is not disturbed by the dry pass
    conv = gpu.convert(g, m)
    assert np.array_equal(conv["hist"], hist) and np.array_equal(conv["sym"], syms)
    assert np.array_equal(conv["mem"].view(np.uint32), mem_o.view(np.uint32))


def test_many_chunks_per_block_and_layer_changes():
    """Enough chunks that blocks take them in groups, layers of very different length, ten clients."""
    sizes = [700_000, 64, 1_300_000, 4096, 10, 250_000]
    fmts = [fmt_tuple(4, 3, scale_for(4, 3, 1.0, 1e-3)[0]), fmt_tuple(2, 1, 900.0), fmt_tuple(5, 2, 3000.0),
            fmt_tuple(4, 3, 100.0), fmt_tuple(3, 0, 500.0), fmt_tuple(2, 1, 1500.0)]
    case = Case(sizes, fmts, n_clients=10, decay=0.7)
    g = np.stack([gennorm(case.n_elem, 1.0, 1e-3, seed=400 + u).numpy() for u in range(10)])
    m = np.stack([gennorm(case.n_elem, 2.0, 1e-4, seed=450 + u).numpy() for u in range(10)])
    gpu = Gpu(case)
    hist, res = _dry(case, gpu, g, m)
    syms, _, nsat, _ = oracle_convert(case, g, m.copy())
    assert np.array_equal(hist, oracle_hist(case, syms)) and np.array_equal(res["n_saturated"], nsat)


def test_argument_checks():
    case = Case([4096], [fmt_tuple(4, 3)], n_clients=1)
    gpu = Gpu(case)
    g = torch.zeros(4100, dtype=torch.float32, device="cuda")
    hist = torch.zeros(256, dtype=torch.int64, device="cuda")
    args = (0.9, gpu.fmts, gpu.segs, 1, 4096, 1, 4096)
    assert co3.co3_histogram(g, g, *args, hist, gpu.res, gpu.ws) == co3.OK
    assert co3.co3_histogram(g[1:], g, *args, hist, gpu.res, gpu.ws) == co3.ERR_INVALID_ARG
    assert co3.co3_histogram(g, g, *args, hist, gpu.res, gpu.ws[:512]) == co3.ERR_CAPACITY
    assert co3.binding._load().co3_histogram(g.data_ptr(), g.data_ptr(), 0.9, gpu.fmts.data_ptr(), gpu.segs.data_ptr(), 1,
                                             4096, 1, 4096, None, gpu.res.data_ptr(), gpu.ws.data_ptr(), gpu.ws.numel(),
                                             None) == co3.ERR_INVALID_ARG
    torch.cuda.synchronize()
