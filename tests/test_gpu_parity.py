"""CUDA path vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, fmt_tuple, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits

pytestmark = pytest.mark.gpu

FORMATS = [(2, 1), (3, 0), (4, 3), (5, 2)]


def _grads(case, seed, beta=1.0, alpha=1e-3):
    g = np.zeros((case.n_clients, case.n_elem), dtype=np.float32)
    for u in range(case.n_clients):
        g[u] = gennorm(case.n_elem, beta, alpha, seed=seed + 1000 * u).numpy()
    return g


def _special_values(fmt):
    """Zeros, sub-normal fp32, every level, every midpoint and its fp32 neighbours, saturating and non-finite."""
    _, lv = oracle.levels(fmt)
    s = np.float32(fmt.scale)
    mids = ((lv[1:] + lv[:-1]) / 2)
    base = np.concatenate([lv, mids]).astype(np.float64) / float(s)
    x = base.astype(np.float32)
    x = np.concatenate([x, np.nextafter(x, np.float32(np.inf)), np.nextafter(x, np.float32(0)),
                        np.nextafter(np.nextafter(x, np.float32(np.inf)), np.float32(np.inf))])
    extra = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, 3e38, -3e38, np.inf, -np.inf, np.nan, 1e30, -1e30],
                     dtype=np.float32)
    x = np.concatenate([x, -x, extra])
    return x.astype(np.float32)


@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("flush", [False, True])
def test_convert_special_values(E, M, flush):
    for scale in (1.0, 1.37, 5317.4585, 2.0 ** -9):
        ft = fmt_tuple(E, M, scale, flush)
        ofmt = oracle.Fmt(E, M, int(flush), ft[3], ft[4])
        x = _special_values(ofmt)
        case = Case([x.size], [ft], 1, decay=0.0)
        grads = x[None, :].copy()
        mems_o = np.zeros_like(grads)
        syms, ghats, nsat, nnf = oracle_convert(case, grads, mems_o)
        out = Gpu(case).convert(grads, np.zeros_like(grads))
        assert out["status"] == co3.OK
        assert np.array_equal(out["sym"], syms)
        assert same_bits(out["mem"], mems_o)
        assert out["res"][0]["n_saturated"] == nsat[0] and out["res"][0]["n_nonfinite"] == nnf[0]
        assert out["res"][0]["status"] == (co3.ERR_NONFINITE if nnf[0] else co3.OK)
        assert np.array_equal(out["hist"], oracle_hist(case, syms))


@pytest.mark.parametrize("E,M", FORMATS)
@pytest.mark.parametrize("flush", [False, True])
def test_encode_special_values_through_the_fused_path(E, M, flush):
    """The same values through co3_encode, whole chunks of them (the path that converts and codes in one pass, with
    its own converter for complete chunks): every level, midpoint and fp32 neighbour, then the non-finite ones."""
    for scale, decay in ((1.0, 0.0), (5317.4585, 0.0), (1.37, 0.5)):
        ft = fmt_tuple(E, M, scale, flush)
        ofmt = oracle.Fmt(E, M, int(flush), ft[3], ft[4])
        x = _special_values(ofmt)
        finite = x[np.isfinite(x)]
        reps = -(-6200 // finite.size)
        g = np.concatenate([np.tile(finite, reps), x]).astype(np.float32)[None, :]
        case = Case([g.size], [ft], 1, decay=decay)
        m0 = (gennorm(g.size, 1.0, 1e-3 / scale, seed=77).numpy() * (decay != 0.0)).astype(np.float32)[None, :]
        mem_o = m0.copy()
        syms, ghats, nsat, nnf = oracle_convert(case, g, mem_o)
        codes = oracle_codes(case, oracle_hist(case, syms))
        want = oracle_encode(case, syms, codes)
        out = Gpu(case).encode(g, m0, codes)
        assert out["status"] == co3.OK and out["guard_ok"]
        assert same_bits(out["mem"], mem_o)
        assert np.array_equal(out["streams"][0], want[0][1])
        assert out["res"][0]["n_saturated"] == nsat[0] and out["res"][0]["n_nonfinite"] == nnf[0]


@pytest.mark.parametrize("n", [0, 1, 2, 31, 32, 33, 4095, 4096, 4097, 50001])
def test_convert_sizes_and_rounds(n):
    ft = fmt_tuple(4, 3, *scale_for(4, 3, 1.0, 1e-3)[:1])
    case = Case([n], [ft], n_clients=2, decay=0.9, stride=n + 13)
    gpu = Gpu(case)
    mem_o = np.zeros((2, n), dtype=np.float32)
    mem_g = np.zeros((2, n), dtype=np.float32)
    for rnd in range(3):
        grads = _grads(case, 10 + rnd)
        syms, _, nsat, _ = oracle_convert(case, grads, mem_o)
        out = gpu.convert(grads, mem_g)
        mem_g = out["mem"]
        assert out["status"] == co3.OK and (out["res"]["status"] == co3.OK).all()
        assert np.array_equal(out["sym"], syms)
        assert same_bits(mem_g, mem_o)
        assert np.array_equal(out["res"]["n_saturated"], nsat)
        assert np.array_equal(out["hist"], oracle_hist(case, syms))


def _mixed_case(n_clients, sizes=(5000, 10, 64, 0, 2048, 4099, 1, 130000, 63)):
    fmts = []
    for k, _ in enumerate(sizes):
        E, M = FORMATS[k % 4]
        beta, alpha = 0.6 + 0.1 * (k % 7), 10.0 ** (-4 + 0.25 * k)
        fmts.append(fmt_tuple(E, M, scale_for(E, M, beta, alpha)[0], flush=(k % 5 == 4)))
    return Case(sizes, fmts, n_clients=n_clients, decay=0.9)


def _layered_grads(case, seed):
    g = np.zeros((case.n_clients, case.n_elem), dtype=np.float32)
    for u in range(case.n_clients):
        for k, n in enumerate(case.sizes):
            beta, alpha = 0.6 + 0.1 * (k % 7), 10.0 ** (-4 + 0.25 * k)
            a = case.offsets[k]
            g[u, a:a + n] = gennorm(n, beta, alpha, seed=seed + 977 * u + k).numpy()
    return g


@pytest.mark.parametrize("n_clients", [1, 3])
def test_encode_streams_bit_identical(n_clients):
    """Fused client pipeline over several rounds: streams, memory and counters equal the oracle's."""
    case = _mixed_case(n_clients)
    gpu = Gpu(case)
    mem_o = np.zeros((n_clients, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    codes = None
    for rnd in range(3):
        grads = _layered_grads(case, 100 * rnd)
        m_before = mem_o.copy()
        syms, _, nsat, _ = oracle_convert(case, grads, mem_o)
        if codes is None:                                   # fitted once, reused afterwards
            codes = oracle_codes(case, oracle_hist(case, syms))
        want = oracle_encode(case, syms, codes)
        out = gpu.encode(grads, mem_g, codes)
        mem_g = out["mem"]
        assert out["status"] == co3.OK and out["guard_ok"]
        assert (out["res"]["status"] == co3.OK).all()
        assert same_bits(mem_g, mem_o)
        for u in range(n_clients):
            st, s = want[u]
            assert st == oracle.OK
            assert out["res"][u]["container_bytes"] == s.size
            assert np.array_equal(out["streams"][u], s)
            ln = np.concatenate([oracle.code_arrays(codes[k])[0][syms[u, case.offsets[k]:case.offsets[k + 1]]]
                                 for k in range(case.n_seg)])
            assert out["res"][u]["payload_bits"] == int(ln.astype(np.int64).sum())
            assert out["res"][u]["n_saturated"] == nsat[u]
        # the symbol path produces the same container
        out2 = gpu.encode(None, None, codes, from_sym=syms)
        assert out2["status"] == co3.OK
        for u in range(n_clients):
            assert np.array_equal(out2["streams"][u], want[u][1])
        del m_before


@pytest.mark.parametrize("n_clients", [1, 2, 3, 4, 5, 8, 10, 16, 17, 20, 21, 35, 41])
def test_decode_aggregate_matches_oracle(n_clients):
    case = _mixed_case(n_clients, sizes=(3000, 10, 64, 0, 2048, 4099, 1, 40000, 63))
    grads = _layered_grads(case, 5)
    mem = np.zeros_like(grads)
    syms, ghats, _, _ = oracle_convert(case, grads, mem)
    codes = oracle_codes(case, oracle_hist(case, syms))
    streams = [s for _, s in oracle_encode(case, syms, codes)]
    st, avg = oracle.decode_aggregate(streams, case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
    assert st == oracle.OK
    gpu = Gpu(case, enc_clients=0)
    out = gpu.decode_aggregate(streams, codes)
    assert out["status"] == co3.OK and out["res"][0]["status"] == co3.OK
    assert same_bits(out["avg"][:case.n_elem], avg)
    assert (out["avg"][case.n_elem:] == -77.0).all()
    # single-stream decode: symbols and values
    d = gpu.decode(streams[0], codes)
    assert d["status"] == co3.OK and d["res"][0]["status"] == co3.OK
    assert np.array_equal(d["sym"][:case.n_elem], syms[0]) and same_bits(d["ghat"][:case.n_elem], ghats[0])
    assert (d["sym"][case.n_elem:] == 0xEE).all()


def test_end_to_end_gpu_only_round_trip_matches_oracle():
    """GPU encode -> GPU decode-aggregate against the oracle's whole pipeline, 4 clients, 2 rounds."""
    case = _mixed_case(4)
    gpu = Gpu(case)
    mem_o = np.zeros((4, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    codes = None
    for rnd in range(2):
        grads = _layered_grads(case, 300 + rnd)
        syms, ghats, _, _ = oracle_convert(case, grads, mem_o)
        if codes is None:
            codes = oracle_codes(case, oracle_hist(case, syms))
        out = gpu.encode(grads, mem_g, codes)
        mem_g = out["mem"]
        agg = gpu.decode_aggregate(out["streams"], codes)
        st, avg = oracle.decode_aggregate([s for _, s in oracle_encode(case, syms, codes)], case.sizes,
                                          [case.ofmt(k) for k in range(case.n_seg)], codes)
        assert agg["res"][0]["status"] == co3.OK and same_bits(agg["avg"][:case.n_elem], avg)
