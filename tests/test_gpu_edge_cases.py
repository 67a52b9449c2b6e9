"""Degenerate and hostile inputs through the C ABI (needs a B200): the results that exist must equal the
oracle's, the others must come back as a status — never as a fault or a hang."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, fmt_tuple, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits

pytestmark = pytest.mark.gpu


def _round_trip(case, grads, codes=None, weights=None):
    """Oracle and GPU encode + decode of one round from zero memory; asserts identity everywhere."""
    mem_o = np.zeros_like(grads)
    syms, ghats, nsat, nnf = oracle_convert(case, grads, mem_o)
    if codes is None:
        hist = oracle_hist(case, syms) if weights is None else weights
        codes = oracle_codes(case, hist)
    want = oracle_encode(case, syms, codes)
    gpu = Gpu(case)
    out = gpu.encode(grads, np.zeros_like(grads), codes)
    assert out["status"] == co3.OK and out["guard_ok"]
    for u in range(case.n_clients):
        assert want[u][0] == oracle.OK
        assert np.array_equal(out["streams"][u], want[u][1])
        assert out["res"][u]["n_saturated"] == nsat[u] and out["res"][u]["n_nonfinite"] == nnf[u]
    assert same_bits(out["mem"], mem_o)
    agg = gpu.decode_aggregate(out["streams"], codes)
    st, avg = oracle.decode_aggregate([w[1] for w in want], case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
    assert agg["res"][0]["status"] == co3.OK and same_bits(agg["avg"][:case.n_elem], avg)
    return out, syms


def test_all_zero_gradient_costs_one_symbol_each():
    case = Case([10000, 77], [fmt_tuple(4, 3, 100.0), fmt_tuple(2, 1, 3.0)], n_clients=2)
    out, syms = _round_trip(case, np.zeros((2, case.n_elem), dtype=np.float32))
    assert (syms == 0).all()
    assert (out["res"]["payload_bits"] == case.n_elem).all()            # the zero symbol gets a 1-bit codeword


def test_all_saturating_gradient():
    case = Case([6000], [fmt_tuple(4, 3, 1.0)], n_clients=1)
    x = gennorm(6000, 1.0, 1.0, seed=1).numpy()
    g = (np.sign(x) * (np.abs(x) * 1e6 + 1e3)).astype(np.float32)          # every |g| is beyond the top level 240
    out, syms = _round_trip(case, g[None, :])
    assert out["res"][0]["n_saturated"] == 6000 and set(np.unique(syms)) <= {0x77, 0xF7}


def test_uniform_symbols_maximum_entropy():
    """Every valid symbol equally often under a flat code: the longest payload per element."""
    fmt = oracle.make_fmt(5, 2, 1.0)
    valid = [s for s in range(256) if oracle.symbol_valid(fmt, s)]
    vals = np.array([oracle.symbol_value(fmt, s) for s in valid], dtype=np.float32)
    rng = np.random.default_rng(0)
    g = vals[rng.integers(0, len(valid), size=50000)]
    case = Case([g.size], [fmt_tuple(5, 2, 1.0)], n_clients=1, decay=0.0)
    out, _ = _round_trip(case, g[None, :], weights=np.ones((1, 256), dtype=np.uint64))
    assert out["res"][0]["payload_bits"] >= 7 * g.size


def _skewed_case():
    """Zero at one bit, codeword lengths up to the 16-bit limit; every valid symbol occurs."""
    fmt = oracle.make_fmt(4, 3, 1.0)
    valid = [s for s in range(256) if oracle.symbol_valid(fmt, s)]
    w = np.zeros((1, 256), dtype=np.uint64)
    for i, s in enumerate(valid):
        w[0, s] = max(1, 2 ** 40 >> (i // 4))                 # four symbols per halving: deep tree, limit applies
    w[0, 0] = 2 ** 44
    n = 300000
    rng = np.random.default_rng(5)
    sym = np.zeros(n, dtype=np.int64)
    idx = rng.choice(n, size=4 * len(valid), replace=False)
    sym[idx] = np.tile(valid, 4)
    vals = np.array([oracle.symbol_value(fmt, s) if oracle.symbol_valid(fmt, s) else 0 for s in range(256)], dtype=np.float32)
    return w, vals[sym]


def test_one_dominant_symbol_and_rare_long_codewords():
    """A skewed stream: zero at one bit, rare symbols at the 16-bit limit (second-level decode tables)."""
    w, g = _skewed_case()
    case = Case([g.size], [fmt_tuple(4, 3, 1.0)], n_clients=3, decay=0.0)
    codes = oracle_codes(case, w)
    ln, _ = oracle.code_arrays(codes[0])
    assert ln.max() == oracle.MAX_CODE_LEN and ln[0] == 1 and (ln > 12).sum() > 20
    grads = np.stack([np.roll(g, 7 * u) for u in range(3)])
    out, syms = _round_trip(case, grads, codes=codes)
    assert len(np.unique(syms)) == 239


def test_tiny_and_unaligned_layers():
    sizes = [10, 64, 1, 3, 2047, 2049, 5, 128]
    fmts = [fmt_tuple(4, 3, scale_for(4, 3, 1.0, 1e-3)[0])] * len(sizes)
    case = Case(sizes, fmts, n_clients=2, stride=sum(sizes) + 3)        # odd stride: nothing is 16-byte aligned
    g = np.stack([gennorm(case.n_elem, 1.0, 1e-3, seed=40 + u).numpy() for u in range(2)])
    _round_trip(case, g)


def test_capacity_too_small_reports_and_writes_nothing_beyond():
    case = Case([40000], [fmt_tuple(4, 3, scale_for(4, 3, 1.0, 1e-3)[0])], n_clients=2)
    g = np.stack([gennorm(40000, 1.0, 1e-3, seed=50 + u).numpy() for u in range(2)])
    mem = np.zeros_like(g)
    syms, _, _, _ = oracle_convert(case, g, mem)
    codes = oracle_codes(case, oracle_hist(case, syms))
    need = oracle_encode(case, syms, codes)[0][1].size
    gpu = Gpu(case)
    cap = (need - 4096) // 16 * 16
    out = gpu.encode(g, np.zeros_like(g), codes, capacity=cap)
    assert out["status"] == co3.OK and out["guard_ok"]
    assert (out["res"]["status"] == co3.ERR_CAPACITY).all()
    assert (out["res"]["container_bytes"] > cap).all()                  # the size it would have needed
    # below the fixed part the host refuses at once
    out = gpu.encode(g, np.zeros_like(g), codes, capacity=256)
    assert out["status"] == co3.ERR_CAPACITY


def test_symbol_without_codeword():
    case = Case([5000], [fmt_tuple(4, 3, scale_for(4, 3, 1.0, 1e-3)[0])], n_clients=2)
    g = np.stack([gennorm(5000, 1.0, 1e-3, seed=60 + u).numpy() for u in range(2)])
    g[1, :] = 0.0                                                      # client 1 only sends zeros
    mem = np.zeros_like(g)
    syms, _, _, _ = oracle_convert(case, g, mem)
    codes = oracle_codes(case, oracle_hist(case, syms))
    ln, bits = oracle.code_arrays(codes[0])
    victim = int(syms[0, np.flatnonzero(syms[0])[0]])
    ln[victim] = 0
    broken = [oracle.make_code(ln, bits)]
    assert oracle.encode(syms[0], case.sizes, broken)[0] == oracle.ERR_NO_CODEWORD
    out = Gpu(case).encode(g, np.zeros_like(g), broken)
    assert out["res"][0]["status"] == co3.ERR_NO_CODEWORD and out["res"][0]["first_bad_chunk"] < 3
    assert out["res"][1]["status"] == co3.OK                           # the other client is unaffected
    assert np.array_equal(out["streams"][1], oracle.encode(syms[1], case.sizes, broken)[1])


def test_invalid_descriptors_are_refused_on_the_device():
    g = gennorm(4096, 1.0, 1e-3, seed=1).numpy()[None, :]
    for bad in [(1, 3, 0, 1.0, 1.0), (4, 4, 0, 1.0, 1.0), (4, 3, 4, 1.0, 1.0), (4, 3, 0, 0.0, 1.0),
                (4, 3, 0, float("inf"), 1.0), (4, 3, 0, 1.0, float("nan")), (7, 0, 0, 1.0, 3e38)]:
        case = Case([4096], [bad], n_clients=1)
        out = Gpu(case).convert(g, np.zeros_like(g))
        assert out["status"] == co3.OK and out["res"][0]["status"] == co3.ERR_INVALID_ARG, bad
        assert same_bits(out["mem"], np.zeros_like(g))                 # nothing was touched
    # segments that do not tile the vector
    case = Case([2000, 2096], [fmt_tuple(4, 3)] * 2, n_clients=1)
    gpu = Gpu(case)
    segs = co3.make_segs(case.sizes)
    segs[1]["elem_off"] = 1999
    gpu.segs = co3.to_device(segs)
    assert gpu.convert(g, np.zeros_like(g))["res"][0]["status"] == co3.ERR_INVALID_ARG
    segs = co3.make_segs([2000, 2000])
    gpu.segs = co3.to_device(segs)
    assert gpu.convert(g, np.zeros_like(g))["res"][0]["status"] == co3.ERR_INVALID_ARG
    # an over-subscribed (not prefix-free) code
    case = Case([4096], [fmt_tuple(4, 3)], n_clients=1)
    ln = np.zeros(256, dtype=int)
    ln[:8] = 2
    out = Gpu(case).encode(g, np.zeros_like(g), [oracle.make_code(ln, np.arange(256) % 4)])
    assert out["res"][0]["status"] == co3.ERR_INVALID_ARG
    # tables whose Kraft sum is at most 1 but in which one codeword starts another ("0" and "01"), or repeats it
    for lens, words in (([1, 2], [0, 1]), ([3, 3, 2], [5, 5, 0]), ([2, 5, 3], [1, 0b01101, 0b100])):
        ln = np.zeros(256, dtype=int)
        bits = np.zeros(256, dtype=int)
        ln[:len(lens)] = lens
        bits[:len(lens)] = words
        assert sum(2.0 ** -l for l in lens) <= 1.0
        out = Gpu(case).encode(g, np.zeros_like(g), [oracle.make_code(ln, bits)])
        assert out["res"][0]["status"] == co3.ERR_INVALID_ARG, (lens, words)
        assert same_bits(out["mem"], np.zeros_like(g))


def test_host_side_argument_checks():
    case = Case([4096], [fmt_tuple(4, 3)], n_clients=1)
    gpu = Gpu(case)
    g = torch.zeros(4100, dtype=torch.float32, device="cuda")
    m = torch.zeros(4100, dtype=torch.float32, device="cuda")
    args = (0.9, gpu.fmts, gpu.segs, 1, 4096, 1, 4096, None, None, gpu.res)
    assert co3.co3_convert(g[1:], m, *args, gpu.ws) == co3.ERR_INVALID_ARG           # misaligned gradient
    assert co3.co3_convert(g, m, *args, gpu.ws[:1024]) == co3.ERR_CAPACITY           # workspace too small
    assert co3.co3_convert(g, m, *args, gpu.ws[1:]) == co3.ERR_INVALID_ARG           # misaligned workspace
    assert co3.co3_convert(g, m, 0.9, gpu.fmts, gpu.segs, 1, 4096, 0, 4096, None, None, gpu.res, gpu.ws) == co3.ERR_INVALID_ARG


@pytest.mark.parametrize("n_clients", [1, 3, 20])
def test_corrupt_streams_are_reported_not_followed(n_clients):
    case = Case([30000, 500], [fmt_tuple(4, 3, scale_for(4, 3, 1.0, 1e-3)[0]), fmt_tuple(2, 1, 300.0)],
                n_clients=n_clients)
    g = np.stack([gennorm(case.n_elem, 1.0, 1e-3, seed=70 + u).numpy() for u in range(n_clients)])
    mem = np.zeros_like(g)
    syms, _, _, _ = oracle_convert(case, g, mem)
    codes = oracle_codes(case, oracle_hist(case, syms))
    streams = [s for _, s in oracle_encode(case, syms, codes)]
    gpu = Gpu(case, enc_clients=0)
    good = gpu.decode_aggregate(streams, codes)
    assert good["res"][0]["status"] == co3.OK
    rng = np.random.default_rng(3)
    hdr_fields = [0, 4, 8, 12, 16, 24, 32, 40, 56]
    victim = n_clients - 1
    for trial in range(12):
        bad = [s.copy() for s in streams]
        b = bad[victim]
        if trial < len(hdr_fields):
            b[hdr_fields[trial]] ^= 0x10                                # header fields
        elif trial == 9:
            off = 64 + 48 + 8                                           # a chunk offset far out of range
            b[off:off + 8] = 0xFF
        elif trial == 10:
            off = 64 + 48 + 8 * 18                                      # sub-chunk offsets
            b[off + 16 * 2 + 2: off + 16 * 2 + 4] = 0xFF
        else:
            pos = rng.integers(b.size - 3000, b.size - 16)              # payload bits
            b[pos] ^= 0xFF
        out = gpu.decode_aggregate(bad, codes)
        if trial < 11:
            assert out["res"][0]["status"] == co3.ERR_CORRUPT, trial
        else:   # flipped payload bits: lengths no longer add up, or (same-length codewords) other values come out
            assert out["res"][0]["status"] == co3.ERR_CORRUPT or not same_bits(out["avg"], good["avg"])
    # truncated readable size
    assert gpu.decode(streams[0], codes, stream_bytes=(streams[0].size // 2) // 16 * 16)["res"][0]["status"] == co3.ERR_CORRUPT
    # afterwards the library still works
    assert gpu.decode_aggregate(streams, codes)["res"][0]["status"] == co3.OK
