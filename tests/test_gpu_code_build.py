"""Huffman tables built on the device (co3_code_build_device) against the oracle's construction
(Sec. IV-A (ii)): every length and every codeword must be identical, for histograms of real conversions,
for weight patterns that exercise the tie order and the length limit, and for every format family.
Needs a B200."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from paper_2204_08211_b200 import binding as B
from co3_inputs import gennorm, scale_for
from harness import fmt_tuple

pytestmark = pytest.mark.gpu


def _device_build(weights: np.ndarray, fmts):
    """weights uint64[n_seg][256], fmts list of fmt tuples -> (status, len[n_seg][256], bits[n_seg][256])."""
    n_seg = len(fmts)
    w = torch.from_numpy(np.ascontiguousarray(weights, dtype=np.uint64).view(np.int64).reshape(-1)).cuda()
    f = B.to_device(B.make_fmts(fmts))
    codes = torch.full((n_seg * B.CODE_DTYPE.itemsize,), 0xAB, dtype=torch.uint8, device="cuda")
    res = torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    st = co3.co3_code_build_device(w, f, n_seg, codes, res)
    assert st == co3.OK
    torch.cuda.synchronize()
    out = np.frombuffer(codes.cpu().numpy().tobytes(), dtype=B.CODE_DTYPE)
    return int(B.read_results(res, 1)[0]["status"]), out["len"].copy(), out["bits"].copy()


def _oracle_build(weights_row, fmt):
    E, M, fl, s, inv = fmt
    code = oracle.code_build(weights_row, oracle.Fmt(E, M, int(fl & 1), s, inv))
    lens, bits = oracle.code_arrays(code)
    return lens, bits


def _check_same(weights, fmts):
    st, lens, bits = _device_build(weights, fmts)
    assert st == co3.OK
    for k, fmt in enumerate(fmts):
        want_len, want_bits = _oracle_build(weights[k], fmt)
        assert np.array_equal(lens[k], want_len), "lengths of segment %d" % k
        assert np.array_equal(bits[k].astype(np.uint32), want_bits), "codewords of segment %d" % k


FORMATS = [fmt_tuple(2, 1, 1.0), fmt_tuple(3, 0, 1.0), fmt_tuple(4, 3, 1.0), fmt_tuple(5, 2, 1.0),
           fmt_tuple(4, 3, 1.0, flush=True), fmt_tuple(2, 5, 7.0), fmt_tuple(6, 1, 0.25, flush=True)]


def test_histograms_of_converted_gradients():
    rng = np.random.default_rng(11)
    fmts, rows = [], []
    for i, (E, M) in enumerate([(4, 3), (2, 1), (5, 2), (3, 0), (4, 3), (4, 3)]):
        beta = [0.5, 1.0, 2.0, 1.5, 0.8, 1.0][i]
        s, inv = scale_for(E, M, beta, 1e-3)
        fmt = (E, M, 0, s, inv)
        g = gennorm(200_000, beta, 1e-3, 1000 + i, "cpu").numpy()
        sym = oracle.convert(g, np.zeros_like(g), 0.0, oracle.Fmt(E, M, 0, s, inv))["sym"]
        fmts.append(fmt)
        rows.append(oracle.histogram(sym))
    _check_same(np.stack(rows), fmts)


def test_weight_patterns_for_ties_and_zero_counts():
    rng = np.random.default_rng(5)
    rows, fmts = [], []
    for fmt in FORMATS:
        rows.append(np.zeros(256, dtype=np.uint64)); fmts.append(fmt)                       # all weights raised to 1
        rows.append(np.full(256, 12345, dtype=np.uint64)); fmts.append(fmt)                 # all equal
        rows.append(rng.integers(0, 4, 256).astype(np.uint64)); fmts.append(fmt)            # many ties
        rows.append(rng.integers(0, 1 << 40, 256).astype(np.uint64)); fmts.append(fmt)      # wide range
        rows.append((np.uint64(1) << rng.integers(0, 30, 256).astype(np.uint64))); fmts.append(fmt)  # powers of two
    _check_same(np.stack(rows), fmts)


def test_length_limit_halves_the_weights():
    # Fibonacci-like weights give a maximally skewed tree, far deeper than 16 levels for the 8-bit formats
    fib = [1, 1]
    while len(fib) < 256:
        fib.append(min(fib[-1] + fib[-2], (1 << 54)))
    rows, fmts = [], []
    for fmt in FORMATS:
        rows.append(np.array(fib, dtype=np.uint64)); fmts.append(fmt)
        rows.append(np.array(fib[::-1], dtype=np.uint64)); fmts.append(fmt)
        w = np.ones(256, dtype=np.uint64); w[0] = 1 << 62                                   # one giant, sum still < 2^63
        rows.append(w); fmts.append(fmt)
    st, lens, bits = _device_build(np.stack(rows), fmts)
    assert st == co3.OK and lens.max() <= co3.MAX_CODE_LEN
    _check_same(np.stack(rows), fmts)


def test_many_segments_in_one_call():
    rng = np.random.default_rng(77)
    n_seg = 300
    fmts = [FORMATS[k % len(FORMATS)] for k in range(n_seg)]
    w = (rng.gamma(0.3, 1e4, size=(n_seg, 256))).astype(np.uint64)
    _check_same(w, fmts)


def test_bad_inputs_come_back_as_status():
    ok = np.ones((1, 256), dtype=np.uint64)
    st, lens, bits = _device_build(ok, [(1, 3, 0, 1.0, 1.0)])            # exponent field too narrow
    assert st == co3.ERR_INVALID_ARG and not lens.any() and not bits.any()
    st, _, _ = _device_build(ok, [(4, 4, 0, 1.0, 1.0)])                    # more than 8 bits
    assert st == co3.ERR_INVALID_ARG
    st, _, _ = _device_build(ok, [(4, 3, 0, -1.0, 1.0)])                   # negative scale
    assert st == co3.ERR_INVALID_ARG
    big = np.full((1, 256), 1 << 56, dtype=np.uint64)                      # 240 valid symbols x 2^56 >= 2^63
    st, _, _ = _device_build(big, [fmt_tuple(4, 3, 1.0)])
    assert st == co3.ERR_INVALID_ARG
    # one bad layer does not disturb its neighbours
    w = np.ones((3, 256), dtype=np.uint64)
    fmts = [fmt_tuple(4, 3, 1.0), (4, 4, 0, 1.0, 1.0), fmt_tuple(2, 1, 1.0)]
    st, lens, bits = _device_build(w, fmts)
    assert st == co3.ERR_INVALID_ARG and not lens[1].any()
    for k in (0, 2):
        want_len, want_bits = _oracle_build(w[k], fmts[k])
        assert np.array_equal(lens[k], want_len) and np.array_equal(bits[k].astype(np.uint32), want_bits)
    # host-side argument checks
    assert co3.co3_code_build_device(torch.zeros(256, dtype=torch.int64, device="cuda"), B.to_device(B.make_fmts([fmt_tuple(4, 3)])),
                                     0, torch.zeros(768, dtype=torch.uint8, device="cuda"),
                                     torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")) == co3.ERR_INVALID_ARG


def test_fit_on_device_round_trip_matches_oracle():
    """The per-round flow with nothing on the host: convert + histogram -> device code build -> encode the
    symbols -> decode; stream and values equal the oracle's with its own code for the same histogram."""
    from paper_2204_08211_b200.session import Co3Session
    sizes = [50_000, 3_000, 70_001]
    E, M = 4, 3
    fm = []
    for k, beta in enumerate((1.0, 0.6, 2.0)):
        s, inv = scale_for(E, M, beta, 1e-3)
        fm.append((E, M, 0, s, inv))
    sess = Co3Session(sizes, fm, 1, 0.9, "cuda")
    g = np.concatenate([gennorm(n, b, 1e-3, 40 + k, "cpu").numpy() for k, (n, b) in enumerate(zip(sizes, (1.0, 0.6, 2.0)))])
    grads = sess.new_client_buffer(); mems = sess.new_client_buffer()
    grads[:sess.n_elem] = torch.from_numpy(g).cuda()
    sym = torch.zeros(sess.stride, dtype=torch.uint8, device="cuda")
    sess.histogram(grads, mems, sym_out=sym, to_host=False)
    sess.set_codes_from_histogram_device()
    sess.encode_symbols(sym)
    avg = sess.decode_aggregate()
    torch.cuda.synchronize()
    assert sess.fit_result()[0]["status"] == co3.OK
    assert sess.encode_results()[0]["status"] == co3.OK and sess.decode_result()[0]["status"] == co3.OK
    # oracle side
    off, codes, osyms, ghat = 0, [], [], []
    for k, n in enumerate(sizes):
        ofmt = oracle.Fmt(E, M, 0, fm[k][3], fm[k][4])
        conv = oracle.convert(g[off:off + n], np.zeros(n, dtype=np.float32), 0.9, ofmt)
        codes.append(oracle.code_build(oracle.histogram(conv["sym"]), ofmt))
        osyms.append(conv["sym"]); ghat.append(conv["ghat"])
        off += n
    st, want = oracle.encode(np.concatenate(osyms), sizes, codes)
    assert st == oracle.OK
    assert np.array_equal(sess.stream_bytes(0), want)
    assert np.array_equal(avg[:sess.n_elem].cpu().numpy().view(np.uint32), np.concatenate(ghat).view(np.uint32))
