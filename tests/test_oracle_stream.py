"""Pins for the oracle's bit packing, container and decode/average (no GPU)."""
import os
import struct

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "stream_example.txt")


def _simple_code():
    lens = np.zeros(256, dtype=int)
    bits = np.zeros(256, dtype=int)
    lens[:4] = [1, 2, 3, 3]
    bits[:4] = [0b0, 0b10, 0b110, 0b111]
    return oracle.make_code(lens, bits)


def _parse(stream, n_seg, C, S):
    hdr = struct.unpack_from("<6I5Q", stream.tobytes(), 0)
    magic, ver, nseg, c, s, _, n_elem, n_chunks, pwords, pbits, total = hdr
    assert magic == int.from_bytes(b"CO3S", "little") and ver == 1 and nseg == n_seg and c == C and s == S
    al = lambda x: (x + 15) & ~15
    seg_off = 64
    chunk_off = al(seg_off + 24 * n_seg)
    sub_off = al(chunk_off + 8 * (n_chunks + 1))
    pay_off = al(sub_off + 2 * n_chunks * (C // S))
    raw = stream.tobytes()
    segs = [struct.unpack_from("<3Q", raw, seg_off + 24 * k) for k in range(n_seg)]
    word_off = list(struct.unpack_from("<%dQ" % (n_chunks + 1), raw, chunk_off))
    subs = list(struct.unpack_from("<%dH" % (n_chunks * (C // S)), raw, sub_off))
    words = list(struct.unpack_from("<%dI" % pwords, raw, pay_off))
    assert total == al(pay_off + 4 * pwords) == len(raw)
    return dict(n_elem=n_elem, n_chunks=n_chunks, payload_bits=pbits, segs=segs, word_off=word_off,
                subs=subs, words=words)


def _bitstring(words, nbits):
    return "".join(format(w, "032b") for w in words)[:nbits]


def test_hand_worked_example():
    g = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        g[k] = v
    sym = np.array([int(x) for x in g["symbols"]], dtype=np.uint8)
    st, stream = oracle.encode(sym, [sym.size], [_simple_code()], chunk_syms=32, sub_syms=8)
    assert st == oracle.OK
    p = _parse(stream, 1, 32, 8)
    assert p["word_off"] == [int(x) for x in g["word_offsets"]]
    assert p["subs"] == [int(x) for x in g["sub_offsets"]]
    assert p["payload_bits"] == int(g["payload_bits"][0]) and p["segs"] == [(37, 0, 76)]
    c0 = "".join(g["chunk0_bits"])
    assert _bitstring(p["words"][0:3], 96) == c0.ljust(96, "0")
    assert _bitstring(p["words"][3:4], 32) == g["chunk1_bits"][0].ljust(32, "0")


@pytest.mark.parametrize("n", [0, 1, 2, 7, 8, 31, 32, 33, 63, 64, 65, 200])
def test_concatenation_brute_force(n):
    """The payload of every chunk is the plain concatenation of the codewords of its symbols."""
    rng = np.random.default_rng(n)
    fmt = oracle.make_fmt(4, 3)
    w = np.zeros(256, dtype=np.uint64)
    valid = [s for s in range(256) if oracle.symbol_valid(fmt, s)]
    w[valid] = (rng.pareto(1.0, size=len(valid)) * 20 + 1).astype(np.uint64)
    code = oracle.code_build(w, fmt)
    ln, bits = oracle.code_arrays(code)
    sym = rng.choice(valid, size=n, p=w[valid] / w[valid].sum()).astype(np.uint8)
    C, S = 32, 8
    st, stream = oracle.encode(sym, [n], [code], chunk_syms=C, sub_syms=S)
    assert st == oracle.OK
    p = _parse(stream, 1, C, S)
    assert p["n_elem"] == n and p["n_chunks"] == (n + C - 1) // C
    total = 0
    for c in range(p["n_chunks"]):
        part = sym[c * C:(c + 1) * C]
        want = "".join(format(int(bits[s]), "0%db" % ln[s]) for s in part)
        w0, w1 = p["word_off"][c], p["word_off"][c + 1]
        assert w1 - w0 == (len(want) + 31) // 32
        assert _bitstring(p["words"][w0:w1], 32 * (w1 - w0)) == want.ljust(32 * (w1 - w0), "0")
        for j in range(C // S):
            off = sum(int(ln[s]) for s in part[:j * S])
            assert p["subs"][c * (C // S) + j] == off
        total += len(want)
    assert p["payload_bits"] == total == int(ln[sym].astype(np.int64).sum())     # r = sum of codeword lengths
    st, sym2, _ = oracle.decode(stream, [n], [fmt], [code], chunk_syms=C, sub_syms=S)
    assert st == oracle.OK and np.array_equal(sym2, sym)


def _multi_segment_case(seed, sizes, C=64, S=16):
    from co3_inputs import gennorm, scale_for
    fmts, codes, syms, ghats = [], [], [], []
    for k, n in enumerate(sizes):
        beta, alpha = 0.7 + 0.1 * k, 10.0 ** (-3 + 0.3 * k)
        E, M = [(4, 3), (2, 1), (5, 2), (3, 0)][k % 4]
        s, inv = scale_for(E, M, beta, alpha)
        fmt = oracle.Fmt(E, M, 0, s, inv)
        g = gennorm(n, beta, alpha, seed=seed * 100 + k).numpy()
        res = oracle.convert(g, np.zeros_like(g), 0.0, fmt)
        fmts.append(fmt)
        codes.append(oracle.code_build(oracle.histogram(res["sym"]), fmt))
        syms.append(res["sym"])
        ghats.append(res["ghat"])
    return fmts, codes, np.concatenate(syms), np.concatenate(ghats)


def test_multi_segment_round_trip_and_tables():
    sizes = [130, 0, 64, 1, 1000, 63]
    C, S = 64, 16
    fmts, codes, sym, ghat = _multi_segment_case(1, sizes, C, S)
    st, stream = oracle.encode(sym, sizes, codes, chunk_syms=C, sub_syms=S)
    assert st == oracle.OK
    p = _parse(stream, len(sizes), C, S)
    first = 0
    for k, n in enumerate(sizes):
        assert p["segs"][k][0] == n and p["segs"][k][1] == first
        first += (n + C - 1) // C
    assert p["n_chunks"] == first and sum(s[2] for s in p["segs"]) == p["payload_bits"]
    assert p["word_off"][0] == 0 and all(b >= a for a, b in zip(p["word_off"], p["word_off"][1:]))
    st, sym2, ghat2 = oracle.decode(stream, sizes, fmts, codes, chunk_syms=C, sub_syms=S)
    assert st == oracle.OK and np.array_equal(sym2, sym) and np.array_equal(ghat2, ghat)   # lossless


def test_capacity_and_corruption_are_reported():
    sizes = [300]
    fmts, codes, sym, _ = _multi_segment_case(2, sizes)
    st, stream = oracle.encode(sym, sizes, codes, chunk_syms=64, sub_syms=16)
    assert st == oracle.OK
    assert stream.size <= oracle.stream_capacity_bytes(sizes, 64, 16)
    st, none = oracle.encode(sym, sizes, codes, chunk_syms=64, sub_syms=16, capacity=stream.size - 16)
    assert st == oracle.ERR_CAPACITY and none is None
    bad = stream.copy()
    bad[0] ^= 1
    assert oracle.decode(bad, sizes, fmts, codes, 64, 16)[0] == oracle.ERR_CORRUPT
    assert oracle.decode(stream[:-16], sizes, fmts, codes, 64, 16)[0] == oracle.ERR_CORRUPT
    rng = np.random.default_rng(0)
    detected = 0
    for _ in range(50):
        bad = stream.copy()
        bad[rng.integers(64, stream.size)] ^= 1 << rng.integers(0, 8)
        st, s2, _ = oracle.decode(bad, sizes, fmts, codes, 64, 16)
        detected += (st == oracle.ERR_CORRUPT) or not np.array_equal(s2, sym)
    assert detected >= 45          # a flipped padding bit changes nothing; everything else must show
    # a symbol without a codeword cannot be encoded
    lens, bits = oracle.code_arrays(codes[0])
    lens[int(sym[0])] = 0
    st, _ = oracle.encode(sym, sizes, [oracle.make_code(lens, bits)], chunk_syms=64, sub_syms=16)
    assert st == oracle.ERR_NO_CODEWORD


def test_decode_aggregate_is_ordered_fp32_mean():
    """(1/U) sum_u ghat^(u): U = 1 returns ghat; equal clients with U a power of two return ghat;
    in general the fp32 running sum in client order divided once by U."""
    sizes = [100, 260]
    C, S = 64, 16
    fmts, codes, sym0, ghat0 = _multi_segment_case(3, sizes, C, S)
    st, s0 = oracle.encode(sym0, sizes, codes, C, S)
    st, avg = oracle.decode_aggregate([s0], sizes, fmts, codes, C, S)
    assert st == oracle.OK and np.array_equal(avg, ghat0)
    st, avg = oracle.decode_aggregate([s0] * 4, sizes, fmts, codes, C, S)
    assert np.array_equal(avg, ghat0)
    # different clients under the same per-layer code
    from co3_inputs import gennorm
    streams, ghats = [], []
    for u in range(5):
        parts, gh = [], []
        off = 0
        for k, n in enumerate(sizes):
            g = gennorm(n, 0.9, 1.0 / fmts[k].scale, seed=900 + 10 * u + k).numpy()
            res = oracle.convert(g, np.zeros_like(g), 0.0, fmts[k])
            parts.append(res["sym"])
            gh.append(res["ghat"])
        st, s = oracle.encode(np.concatenate(parts), sizes, codes, C, S)
        assert st == oracle.OK
        streams.append(s)
        ghats.append(np.concatenate(gh))
    st, avg = oracle.decode_aggregate(streams, sizes, fmts, codes, C, S)
    acc = np.zeros_like(ghats[0])
    for gh in ghats:
        acc = (acc + gh).astype(np.float32)
    assert np.array_equal(avg, (acc / np.float32(5)).astype(np.float32))
    exact = np.mean(np.stack(ghats).astype(np.float64), axis=0)
    assert np.abs(avg - exact).max() <= 4 * 2.0 ** -24 * np.abs(np.stack(ghats)).sum(axis=0).max()
