"""co3_convert_static — the conversion for hosts that cannot allocate device memory — against co3_convert.

Collected last on purpose (file name): a run that stops at the first failure has then already run every
other test.  The entry point keeps its scratch in an array inside the library, so the test calls it twice in
a row (the second call meets the first call's leftovers) with different inputs and layouts and requires both
results to equal what the ordinary entry point, given a caller-owned workspace, produces: symbols, histogram
and counters exactly, the error memory bit for bit (the tolerance of the other parity tests).
"""
import numpy as np
import pytest
import torch

import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for

pytestmark = pytest.mark.gpu


def _run(entry, sizes, fmts, n_clients, seed, decay=0.9):
    n_elem = int(sum(sizes))
    stride = n_elem + 4
    fm = co3.to_device(co3.make_fmts(fmts))
    sg = co3.to_device(co3.make_segs(sizes))
    g = torch.zeros(n_clients * stride, dtype=torch.float32, device="cuda")
    m = torch.zeros_like(g)
    for u in range(n_clients):
        g[u * stride:u * stride + n_elem] = gennorm(n_elem, 0.9, 1e-3, seed=seed + u).cuda()
        m[u * stride:u * stride + n_elem] = gennorm(n_elem, 1.5, 1e-4, seed=seed + 50 + u).cuda()
    sym = torch.full((n_clients * stride,), 0xEE, dtype=torch.uint8, device="cuda")
    hist = torch.full((len(sizes) * 256,), 5, dtype=torch.int64, device="cuda")
    res = torch.zeros(n_clients * co3.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    st = entry(g, m, decay, fm, sg, len(sizes), n_elem, n_clients, stride, sym, hist, res)
    torch.cuda.synchronize()
    assert st == co3.OK, co3.co3_status_string(st)
    r = co3.read_results(res, n_clients)
    return sym.cpu().numpy(), m.cpu().numpy(), hist.cpu().numpy(), r


def _with_workspace(n_elem, n_seg):
    ws = torch.empty(co3.co3_workspace_bytes(n_elem, n_seg, 0), dtype=torch.uint8, device="cuda")

    def entry(g, m, decay, fm, sg, n_seg_, n_elem_, n_clients, stride, sym, hist, res):
        return co3.co3_convert(g, m, decay, fm, sg, n_seg_, n_elem_, n_clients, stride, sym, hist, res, ws)
    return entry


def test_static_scratch_matches_workspace_entry_point_twice():
    cases = [
        ([5000, 10, 64, 0, 2048, 4099, 1, 30000], 2, 11),
        ([70001, 333], 3, 12),                               # a different layout over the same scratch bytes
    ]
    for sizes, n_clients, seed in cases:
        fmts = []
        for k in range(len(sizes)):
            E, M = [(4, 3), (2, 1), (5, 2), (3, 0)][k % 4]
            fmts.append((E, M, 0) + scale_for(E, M, 0.9, 1e-3))
        want = _run(_with_workspace(sum(sizes), len(sizes)), sizes, fmts, n_clients, seed)
        got = _run(co3.co3_convert_static, sizes, fmts, n_clients, seed)
        assert np.array_equal(got[0], want[0])                                   # symbols
        assert np.array_equal(got[1].view(np.uint32), want[1].view(np.uint32))   # error memory, bit for bit
        assert np.array_equal(got[2], want[2])                                   # histogram
        for f in ("status", "n_saturated", "n_nonfinite"):
            assert np.array_equal(got[3][f], want[3][f])
        assert (got[3]["status"] == co3.OK).all()


def test_static_scratch_refuses_layouts_beyond_its_size():
    n_elem = 1 << 30                                          # needs far more than the built-in 2 MiB
    assert co3.co3_workspace_bytes(n_elem, 1, 0) > co3.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    raw = torch.zeros(64, dtype=torch.uint8, device="cuda")
    st = co3.co3_convert_static(dummy, dummy, 0.9, raw, raw, 1, n_elem, 1, n_elem, None, None, raw)
    assert st == co3.ERR_CAPACITY
