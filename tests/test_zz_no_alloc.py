"""co3_convert_static — the conversion for hosts that cannot allocate device memory.

Collected last on purpose (file name): a run that stops at the first failure has then already run every
other test.  The entry point keeps its scratch in an array inside the library, so the test calls it twice in
a row (the second call meets the first call's leftovers) with different inputs and layouts and requires both
results to equal what the ordinary entry point, given a caller-owned workspace, produces, and what the CPU
oracle computes from the same inputs: symbols, histogram and counters exactly, the error memory bit for bit
(the tolerance of the other parity tests).  A last test checks the property in the name: the amount of free
device memory the runtime reports does not move across calls.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import RESNET18_LAYER_SIZES, gennorm, scale_for

pytestmark = pytest.mark.gpu


def _inputs(sizes, n_clients, seed):
    n_elem = int(sum(sizes))
    stride = n_elem + 4
    g = torch.zeros(n_clients * stride, dtype=torch.float32, device="cuda")
    m = torch.zeros_like(g)
    for u in range(n_clients):
        g[u * stride:u * stride + n_elem] = gennorm(n_elem, 0.9, 1e-3, seed=seed + u).cuda()
        m[u * stride:u * stride + n_elem] = gennorm(n_elem, 1.5, 1e-4, seed=seed + 50 + u).cuda()
    return g, m, n_elem, stride


def _run(entry, sizes, fmts, n_clients, seed, decay=0.9):
    g, m, n_elem, stride = _inputs(sizes, n_clients, seed)
    fm = co3.to_device(co3.make_fmts(fmts))
    sg = co3.to_device(co3.make_segs(sizes))
    sym = torch.full((n_clients * stride,), 0xEE, dtype=torch.uint8, device="cuda")
    hist = torch.full((len(sizes) * 256,), 5, dtype=torch.int64, device="cuda")
    res = torch.zeros(n_clients * co3.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    st = entry(g, m, decay, fm, sg, len(sizes), n_elem, n_clients, stride, sym, hist, res)
    torch.cuda.synchronize()
    assert st == co3.OK, co3.co3_status_string(st)
    r = co3.read_results(res, n_clients)
    return sym.cpu().numpy(), m.cpu().numpy(), hist.cpu().numpy(), r


def _oracle_run(sizes, fmts, n_clients, seed, decay=0.9):
    """The same call through the CPU oracle, layer by layer: symbols, new memory, histogram, counters."""
    g, m, n_elem, stride = _inputs(sizes, n_clients, seed)
    g, m = g.cpu().numpy(), m.cpu().numpy()
    sym = np.full(n_clients * stride, 0xEE, dtype=np.uint8)
    hist = np.zeros((len(sizes), 256), dtype=np.int64)
    nsat = np.zeros(n_clients, dtype=np.uint64)
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    for u in range(n_clients):
        for k, (E, M, fl, s, inv) in enumerate(fmts):
            a, b = u * stride + int(offs[k]), u * stride + int(offs[k + 1])
            mk = m[a:b].copy()
            r = oracle.convert(g[a:b].copy(), mk, decay, oracle.Fmt(E, M, fl, s, inv))
            m[a:b] = mk
            sym[a:b] = r["sym"]
            hist[k] += oracle.histogram(r["sym"]).astype(np.int64)
            nsat[u] += r["n_saturated"]
    return sym, m, hist.reshape(-1), nsat


def _with_workspace(n_elem, n_seg):
    ws = torch.empty(co3.co3_workspace_bytes(n_elem, n_seg, 0), dtype=torch.uint8, device="cuda")

    def entry(g, m, decay, fm, sg, n_seg_, n_elem_, n_clients, stride, sym, hist, res):
        return co3.co3_convert(g, m, decay, fm, sg, n_seg_, n_elem_, n_clients, stride, sym, hist, res, ws)
    return entry


def _mixed_fmts(n):
    out = []
    for k in range(n):
        E, M = [(4, 3), (2, 1), (5, 2), (3, 0)][k % 4]
        out.append((E, M, 0) + scale_for(E, M, 0.9, 1e-3))
    return out


def test_static_scratch_matches_workspace_entry_point_and_oracle_twice():
    cases = [
        ([5000, 10, 64, 0, 2048, 4099, 1, 30000], 2, 11),
        ([70001, 333], 3, 12),                               # a different layout over the same scratch bytes
    ]
    for sizes, n_clients, seed in cases:
        fmts = _mixed_fmts(len(sizes))
        want = _run(_with_workspace(sum(sizes), len(sizes)), sizes, fmts, n_clients, seed)
        got = _run(co3.co3_convert_static, sizes, fmts, n_clients, seed)
        ref = _oracle_run(sizes, fmts, n_clients, seed)
        for other in (want, ref):
            assert np.array_equal(got[0], other[0])                                   # symbols
            assert np.array_equal(got[1].view(np.uint32), other[1].view(np.uint32))   # error memory, bit for bit
            assert np.array_equal(got[2], other[2])                                   # histogram
        for f in ("status", "n_saturated", "n_nonfinite"):
            assert np.array_equal(got[3][f], want[3][f])
        assert (got[3]["status"] == co3.OK).all() and np.array_equal(got[3]["n_saturated"], ref[3])


def test_static_scratch_holds_the_62_layer_layout():
    """The largest layout the header promises to fit (62 layers, 11,181,642 elements), against the oracle."""
    sizes = list(RESNET18_LAYER_SIZES)
    assert co3.co3_workspace_bytes(sum(sizes), len(sizes), 0) <= co3.STATIC_SCRATCH_BYTES
    fmts = _mixed_fmts(len(sizes))
    got = _run(co3.co3_convert_static, sizes, fmts, 1, 21)
    ref = _oracle_run(sizes, fmts, 1, 21)
    assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1].view(np.uint32), ref[1].view(np.uint32))
    assert np.array_equal(got[2], ref[2]) and got[3][0]["status"] == co3.OK and got[3][0]["n_saturated"] == ref[3][0]


def test_static_scratch_calls_leave_free_device_memory_unchanged():
    """With every buffer made beforehand and one call done (it looks the array's address up), two more calls must
    not change the free device memory the CUDA runtime reports: nothing was allocated, nothing freed."""
    sizes, n_clients = [50000, 777, 4096], 2
    fmts = _mixed_fmts(len(sizes))
    g, m, n_elem, stride = _inputs(sizes, n_clients, 31)
    fm = co3.to_device(co3.make_fmts(fmts))
    sg = co3.to_device(co3.make_segs(sizes))
    sym = torch.zeros(n_clients * stride, dtype=torch.uint8, device="cuda")
    hist = torch.zeros(len(sizes) * 256, dtype=torch.int64, device="cuda")
    res = torch.zeros(n_clients * co3.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    call = lambda: co3.co3_convert_static(g, m, 0.9, fm, sg, len(sizes), n_elem, n_clients, stride, sym, hist, res)
    assert call() == co3.OK
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    assert call() == co3.OK and call() == co3.OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert (co3.read_results(res, n_clients)["status"] == co3.OK).all()


def test_static_scratch_refuses_layouts_beyond_its_size():
    n_elem = 1 << 30                                          # needs far more than the built-in 2 MiB
    assert co3.co3_workspace_bytes(n_elem, 1, 0) > co3.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    raw = torch.zeros(64, dtype=torch.uint8, device="cuda")
    st = co3.co3_convert_static(dummy, dummy, 0.9, raw, raw, 1, n_elem, 1, n_elem, None, None, raw)
    assert st == co3.ERR_CAPACITY
