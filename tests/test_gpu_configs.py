"""The five workload configurations through the C ABI against the oracle (needs a B200).

Small-scale versions are compared element by element; the full-size launch that bench.py times (config 2:
10 clients x 11,181,642 elements) is compared on sampled chunks, which the oracle can compute one by one
because chunks are coded independently, plus properties that hold at any size.
"""
import numpy as np
import pytest
import torch

import co3_inputs as ci
import oracle
import paper_2204_08211_b200 as co3
from harness import Case, Gpu, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits
from paper_2204_08211_b200.session import Co3Session

pytestmark = pytest.mark.gpu


def _fmts(cfg, sizes, fmt=None):
    E, M = fmt or cfg["fmt"]
    return [(E, M, 0) + ci.scale_for(E, M, cfg["beta"][k % len(cfg["beta"])], cfg["alpha"][k % len(cfg["alpha"])])
            for k in range(len(sizes))]


def _grads(cfg, sizes, n_clients, rnd, outliers=False):
    g = np.zeros((n_clients, sum(sizes)), dtype=np.float32)
    offs = np.concatenate([[0], np.cumsum(sizes)])
    for u in range(n_clients):
        seed = ci.client_round_seed(cfg["seed"], u, rnd)
        for k, n in enumerate(sizes):
            g[u, offs[k]:offs[k + 1]] = ci.gennorm(
                n, cfg["beta"][k % len(cfg["beta"])], cfg["alpha"][k % len(cfg["alpha"])], seed * 1_000_003 + k, "cpu",
                cfg.get("outlier_frac", 0.0) if outliers else 0.0, cfg.get("outlier_mult", 1.0)).numpy()
    return g


def test_config1_code_fitted_every_round():
    """1 client, 1e6 elements, [1,4,3], decay 0.9, 4 of the 10 rounds: convert + histogram -> code -> encode symbols."""
    cfg = ci.config(1)
    sizes = list(cfg["sizes"])
    case = Case(sizes, _fmts(cfg, sizes), n_clients=1, decay=cfg["decay"])
    gpu = Gpu(case)
    mem_o = np.zeros((1, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    for rnd in range(4):
        g = _grads(cfg, sizes, 1, rnd)
        syms, ghats, _, _ = oracle_convert(case, g, mem_o)
        hist = oracle_hist(case, syms)
        conv = gpu.convert(g, mem_g)
        mem_g = conv["mem"]
        assert np.array_equal(conv["sym"], syms) and same_bits(mem_g, mem_o) and np.array_equal(conv["hist"], hist)
        st, code = co3.co3_code_build(conv["hist"][0], co3.make_fmts(case.fmts))          # the library's builder
        ocode = oracle.code_build(hist[0], case.ofmt(0))
        ln, bits = oracle.code_arrays(ocode)
        assert st == co3.OK and np.array_equal(code["len"][0], ln) and np.array_equal(code["bits"][0], bits)
        want = oracle_encode(case, syms, [ocode])[0][1]
        out = gpu.encode(None, None, [ocode], from_sym=syms)
        assert np.array_equal(out["streams"][0], want)
        dec = gpu.decode(out["streams"][0], [ocode])
        assert dec["res"][0]["status"] == co3.OK
        assert np.array_equal(dec["sym"][:case.n_elem], syms[0]) and same_bits(dec["ghat"][:case.n_elem], ghats[0])


def test_config2_layout_two_clients_three_rounds():
    """The 62-layer layout at full length with 2 of the 10 clients: everything compared element by element."""
    cfg = ci.config(2)
    sizes = list(cfg["sizes"])
    case = Case(sizes, _fmts(cfg, sizes), n_clients=2, decay=cfg["decay"])
    gpu = Gpu(case)
    mem_o = np.zeros((2, case.n_elem), dtype=np.float32)
    mem_g = mem_o.copy()
    codes = None
    for rnd in range(3):
        g = _grads(cfg, sizes, 2, rnd)
        syms, _, nsat, _ = oracle_convert(case, g, mem_o)
        if codes is None:
            codes = oracle_codes(case, oracle_hist(case, syms))
        want = oracle_encode(case, syms, codes)
        out = gpu.encode(g, mem_g, codes)
        mem_g = out["mem"]
        assert same_bits(mem_g, mem_o) and np.array_equal(out["res"]["n_saturated"], nsat)
        for u in range(2):
            assert np.array_equal(out["streams"][u], want[u][1])
        agg = gpu.decode_aggregate(out["streams"], codes)
        st, avg = oracle.decode_aggregate([w[1] for w in want], sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
        assert agg["res"][0]["status"] == co3.OK and same_bits(agg["avg"][:case.n_elem], avg)


def test_config3_many_clients_batched():
    """100 clients in one batched encode and one decode-aggregate (layer layout scaled down 64x)."""
    cfg = ci.config(3)
    sizes = [max(1, n // 64) for n in cfg["sizes"]]
    case = Case(sizes, _fmts(cfg, sizes), n_clients=100, decay=cfg["decay"])
    g = _grads(cfg, sizes, 100, 0)
    mem_o = np.zeros_like(g)
    syms, _, _, _ = oracle_convert(case, g, mem_o)
    codes = oracle_codes(case, oracle_hist(case, syms))
    want = oracle_encode(case, syms, codes)
    gpu = Gpu(case)
    out = gpu.encode(g, np.zeros_like(g), codes)
    assert same_bits(out["mem"], mem_o)
    for u in range(100):
        assert np.array_equal(out["streams"][u], want[u][1])
    agg = gpu.decode_aggregate(out["streams"], codes)
    st, avg = oracle.decode_aggregate([w[1] for w in want], sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
    assert agg["res"][0]["status"] == co3.OK and same_bits(agg["avg"][:case.n_elem], avg)


def test_config4_format_shape_decay_sweep():
    """All 36 cells of the sweep at 200k elements, 2 rounds each."""
    cfg = ci.config(4)
    n = 200_000
    for cell in cfg["cells"]:
        E, M = cell["fmt"]
        c = dict(cfg, beta=(cell["beta"],))
        case = Case([n], _fmts(c, [n], (E, M)), n_clients=1, decay=cell["decay"])
        gpu = Gpu(case)
        mem_o = np.zeros((1, n), dtype=np.float32)
        mem_g = mem_o.copy()
        codes = None
        for rnd in range(2):
            g = _grads(c, [n], 1, rnd)
            syms, ghats, nsat, _ = oracle_convert(case, g, mem_o)
            if codes is None:
                codes = oracle_codes(case, oracle_hist(case, syms))
            out = gpu.encode(g, mem_g, codes)
            mem_g = out["mem"]
            assert same_bits(mem_g, mem_o), cell
            assert np.array_equal(out["streams"][0], oracle_encode(case, syms, codes)[0][1]), cell
            assert out["res"][0]["n_saturated"] == nsat[0]
            dec = gpu.decode(out["streams"][0], codes, want_sym=False)
            assert same_bits(dec["ghat"][:n], ghats[0]), cell


def test_config5_outliers_and_eight_clients():
    """GenNorm(0.8) with 0.01 % outliers at 100x scale: 3M elements x 1 client and 400k x 8 clients, 3 rounds."""
    cfg = ci.config(5)
    for n, clients in ((3_000_000, 1), (400_000, 8)):
        case = Case([n], _fmts(cfg, [n]), n_clients=clients, decay=cfg["decay"])
        gpu = Gpu(case)
        mem_o = np.zeros((clients, n), dtype=np.float32)
        mem_g = mem_o.copy()
        codes = None
        for rnd in range(3):
            g = _grads(cfg, [n], clients, rnd, outliers=True)
            syms, _, nsat, _ = oracle_convert(case, g, mem_o)
            if codes is None:
                codes = oracle_codes(case, oracle_hist(case, syms))
            want = oracle_encode(case, syms, codes)
            out = gpu.encode(g, mem_g, codes)
            mem_g = out["mem"]
            assert same_bits(mem_g, mem_o) and np.array_equal(out["res"]["n_saturated"], nsat)
            for u in range(clients):
                assert np.array_equal(out["streams"][u], want[u][1])
            agg = gpu.decode_aggregate(out["streams"], codes)
            st, avg = oracle.decode_aggregate([w[1] for w in want], [n], [case.ofmt(0)], codes)
            assert same_bits(agg["avg"][:n], avg)


def test_long_input_two_level_offsets():
    """35.7 M elements in one layer (beyond 16384 chunks the chunk offsets come from the multi-block scan):
    the whole stream and the decoded values against the oracle."""
    cfg = ci.config(5)
    n = 35_700_003
    case = Case([n], _fmts(cfg, [n]), n_clients=1, decay=cfg["decay"])
    g = _grads(cfg, [n], 1, 0, outliers=True)
    mem_o = np.zeros((1, n), dtype=np.float32)
    syms, ghats, nsat, _ = oracle_convert(case, g, mem_o)
    codes = oracle_codes(case, oracle_hist(case, syms))
    want = oracle_encode(case, syms, codes)[0][1]
    gpu = Gpu(case)
    out = gpu.encode(g, np.zeros_like(g), codes)
    assert out["status"] == co3.OK and out["res"][0]["status"] == co3.OK and out["guard_ok"]
    assert same_bits(out["mem"], mem_o) and out["res"][0]["n_saturated"] == nsat[0]
    assert np.array_equal(out["streams"][0], want)
    dec = gpu.decode(out["streams"][0], codes, want_sym=False)
    assert dec["res"][0]["status"] == co3.OK and same_bits(dec["ghat"][:n], ghats[0])


def test_config2_full_size_sampled_chunks():
    """The launch bench.py times (10 clients x 11,181,642 elements, second round so that memory is live):
    sampled chunks against the oracle, and size-independent properties of the streams."""
    import bench
    cfg, sizes, fmts, clients = bench.workload(2)
    sess = Co3Session(sizes, fmts, clients, cfg["decay"], "cuda")
    g0 = bench.make_grads(cfg, sizes, clients, sess.stride, 0, "cuda")
    g1 = bench.make_grads(cfg, sizes, clients, sess.stride, 1, "cuda")
    mems = sess.new_client_buffer()
    hist = sess.histogram(g0, sess.new_client_buffer())
    assert int(hist.sum()) == sess.n_elem * clients
    sess.set_codes_from_weights(hist)
    sess.encode(g0, mems)
    mem_before = mems.clone()
    sess.encode(g1, mems)
    avg = sess.decode_aggregate().clone()
    torch.cuda.synchronize()
    res = sess.encode_results()
    assert (res["status"] == co3.OK).all() and sess.decode_result()["status"][0] == co3.OK

    C = co3.CHUNK_SYMS
    ofmts = [oracle.Fmt(E, M, 0, s, inv) for (E, M, _, s, inv) in fmts]
    ocodes = [oracle.code_build(hist[k], ofmts[k]) for k in range(len(sizes))]     # the oracle's own tables ...
    for k in range(len(sizes)):                                                    # ... which the library's equal
        ln, bits = oracle.code_arrays(ocodes[k])
        assert np.array_equal(sess.codes_host[k]["len"], ln) and np.array_equal(sess.codes_host[k]["bits"].astype(np.uint32), bits)
    seg_first = np.concatenate([[0], np.cumsum([(n + C - 1) // C for n in sizes])])
    seg_off = np.concatenate([[0], np.cumsum(sizes)])
    n_chunks = int(seg_first[-1])
    al = lambda x: (x + 15) & ~15
    chunk_off = al(64 + 24 * len(sizes))
    sub_off = al(chunk_off + 8 * (n_chunks + 1))
    pay_off = al(sub_off + 32 * n_chunks)
    rng = np.random.default_rng(0)
    picks = sorted(set(int(c) for c in rng.integers(0, n_chunks, size=24)) | {0, n_chunks - 1, int(seg_first[1]) - 1})
    streams = [sess.stream_bytes(u) for u in range(clients)]
    for u in range(clients):
        s = streams[u]
        assert int(s[40:48].view(np.uint64)[0]) * 4 + pay_off <= s.size == res[u]["container_bytes"]
        wo = s[chunk_off:chunk_off + 8 * (n_chunks + 1)].view(np.uint64)
        assert wo[0] == 0 and (np.diff(wo.astype(np.int64)) >= 0).all() and wo[-1] == s[40:48].view(np.uint64)[0]
        segbits = s[64:64 + 24 * len(sizes)].view(np.uint64).reshape(-1, 3)
        assert np.array_equal(segbits[:, 0], np.array(sizes, dtype=np.uint64))
        assert int(segbits[:, 2].sum()) == res[u]["payload_bits"] == int(s[48:56].view(np.uint64)[0])
    for c in picks:
        k = int(np.searchsorted(seg_first, c, side="right") - 1)
        start = (c - int(seg_first[k])) * C
        cnt = min(C, sizes[k] - start)
        lo = int(seg_off[k]) + start
        ghat_sum = None
        for u in range(clients):
            base = u * sess.stride + lo
            g = g1[base:base + cnt].cpu().numpy()
            m = mem_before[base:base + cnt].cpu().numpy().copy()
            r = oracle.convert(g, m, cfg["decay"], ofmts[k])
            assert same_bits(mems[base:base + cnt].cpu().numpy(), m)
            st, want = oracle.encode(r["sym"], [cnt], [ocodes[k]])
            assert st == oracle.OK
            # the oracle's one-chunk stream: its payload and sub-chunk offsets are this chunk's
            w_pay = al(al(al(64 + 24) + 16) + 32)
            s = streams[u]
            wo = s[chunk_off + 8 * c:chunk_off + 8 * c + 16].view(np.uint64)
            nwords = int(want[40:48].view(np.uint64)[0])
            assert int(wo[1] - wo[0]) == nwords
            assert np.array_equal(s[pay_off + 4 * int(wo[0]):pay_off + 4 * int(wo[1])], want[w_pay:w_pay + 4 * nwords])
            assert np.array_equal(s[sub_off + 32 * c:sub_off + 32 * c + 32], want[al(al(64 + 24) + 16):al(al(64 + 24) + 16) + 32])
            gh = r["ghat"]
            ghat_sum = gh.copy() if ghat_sum is None else (ghat_sum + gh).astype(np.float32)
        want_avg = (ghat_sum / np.float32(clients)).astype(np.float32)
        assert same_bits(avg[lo:lo + cnt].cpu().numpy(), want_avg)


# ---------------------------------------------------------------------------------------------- full sizes
def _top_level(E, M):
    """Largest level of the format [1, E, M] before the multiplier: (2 - 2^-M) 2^(2^(E-1)-1), Sec. V-B boundary."""
    return float((2.0 - 2.0 ** -M) * 2.0 ** (2 ** (E - 1) - 1))


def _codes_from_oracle_sample(sess, g0, sizes, ofmts, decay, n_sample=32768):
    """One code per layer computed by the oracle alone: the symbol counts of the leading elements of client 0's
    first-round gradient (zero memory).  Any complete code serves the comparison; this one is close to the fitted one."""
    seg_off = np.concatenate([[0], np.cumsum(sizes)])
    ocodes = []
    for k, n in enumerate(sizes):
        g = g0[int(seg_off[k]):int(seg_off[k]) + min(int(n), n_sample)].cpu().numpy()
        r = oracle.convert(g, np.zeros(g.size, dtype=np.float32), decay, ofmts[k])
        ocodes.append(oracle.code_build(oracle.histogram(r["sym"]), ofmts[k]))
    arr = np.zeros(len(sizes), dtype=co3.CODE_DTYPE)
    for k, c in enumerate(ocodes):
        ln, bits = oracle.code_arrays(c)
        arr[k]["len"] = ln
        arr[k]["bits"] = bits.astype(np.uint16)
    sess.set_codes(arr)
    return ocodes


def _full_size_sampled(cfg, sizes, fmts, clients, n_random=24, payload_clients=8, seed=0):
    """Two rounds of the batched encode and one decode-aggregate at full size through the session (the calls and the
    launch shapes bench.py times), compared with the oracle on sampled chunks: error memory, payload words, sub-chunk
    offsets and the averaged gradient bit for bit; plus properties of whole streams and the saturation counters of
    the first round against a plain fp32 comparison of every element.  Returns what the caller may want to look at."""
    import bench
    C = co3.CHUNK_SYMS
    sess = Co3Session(sizes, fmts, clients, cfg["decay"], "cuda")
    ofmts = [oracle.Fmt(E, M, 0, s, inv) for (E, M, _, s, inv) in fmts]
    g0 = bench.make_grads(cfg, sizes, clients, sess.stride, 0, "cuda")
    ocodes = _codes_from_oracle_sample(sess, g0, sizes, ofmts, cfg["decay"])
    mems = sess.new_client_buffer()
    sess.encode(g0, mems)
    torch.cuda.synchronize()
    res0 = sess.encode_results()
    assert (res0["status"] == co3.OK).all(), res0["status"]
    seg_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    # first round, zero memory: v = g, so an element saturates exactly when |fl32(g * scale)| exceeds the largest level
    n_sat = torch.zeros(clients, dtype=torch.int64, device="cuda")
    g0v = g0.view(clients, sess.stride)
    for k, (E, M, _, s, _) in enumerate(fmts):
        t = g0v[:, int(seg_off[k]):int(seg_off[k + 1])] * np.float32(s)
        n_sat += (t.abs() > _top_level(E, M)).sum(dim=1)
        del t
    assert np.array_equal(n_sat.cpu().numpy().astype(np.uint64), res0["n_saturated"])
    del g0v, g0
    mem_before = mems.clone()
    g1 = bench.make_grads(cfg, sizes, clients, sess.stride, 1, "cuda")
    sess.encode(g1, mems)
    avg = sess.decode_aggregate()
    torch.cuda.synchronize()
    res = sess.encode_results()
    assert (res["status"] == co3.OK).all() and sess.decode_result()["status"][0] == co3.OK

    seg_first = np.concatenate([[0], np.cumsum([(n + C - 1) // C for n in sizes])]).astype(np.int64)
    n_chunks = int(seg_first[-1])
    al = lambda x: (x + 15) & ~15
    chunk_off = al(64 + 24 * len(sizes))
    sub_off = al(chunk_off + 8 * (n_chunks + 1))
    pay_off = al(sub_off + 32 * n_chunks)
    cap = sess.capacity
    sv = sess.streams.view(clients, cap)

    # whole-stream properties, on the first, a middle and the last client
    check_clients = sorted({0, clients // 2, clients - 1})
    wo_last = None
    for u in check_clients:
        head = sv[u, :pay_off].cpu().numpy()
        h32, h64 = head[:64].view(np.uint32), head[:64].view(np.uint64)
        assert h32[0] == 0x53334F43 and h32[1] == 1 and h32[2] == len(sizes) and h32[3] == C and h32[4] == co3.SUB_SYMS
        assert h64[3] == sess.n_elem and h64[4] == n_chunks
        assert h64[6] == res[u]["payload_bits"] and h64[7] == res[u]["container_bytes"] == al(pay_off + 4 * int(h64[5]))
        wo = head[chunk_off:chunk_off + 8 * (n_chunks + 1)].view(np.uint64).astype(np.int64)
        assert wo[0] == 0 and (np.diff(wo) >= 0).all() and (np.diff(wo) <= C * 16 // 32).all() and wo[-1] == h64[5]
        segtab = head[64:64 + 24 * len(sizes)].view(np.uint64).reshape(-1, 3)
        assert np.array_equal(segtab[:, 0], np.array(sizes, dtype=np.uint64))
        assert np.array_equal(segtab[:, 1].astype(np.int64), seg_first[:-1])
        assert int(segtab[:, 2].sum()) == res[u]["payload_bits"]
        # payload bits of a chunk round up to its words: the container holds between bits/32 and bits/32 + chunks words
        assert int(h64[6]) <= 32 * int(h64[5]) < int(h64[6]) + 32 * n_chunks + 32
        wo_last = wo

    # chunks to compare: ends, segment and scan-range boundaries, the chunks around the 2^31-byte and 2^32-bit marks
    # of the inputs and of the payload, and random ones
    rng = np.random.default_rng(seed)
    picks = {0, n_chunks - 1, int(seg_first[1]) - 1, int(seg_first[len(sizes) // 2]), int(seg_first[-2])}
    picks |= {c for c in (4095, 4096, 16383, 16384, 65535, 65536, n_chunks - 4097) if 0 <= c < n_chunks}
    picks |= {int(c) for c in rng.integers(0, n_chunks, size=n_random)}
    for mark_words in (1 << 27, 1 << 29):                       # payload bit 2^32, payload byte 2^31
        c = int(np.searchsorted(wo_last, mark_words, side="right")) - 1
        if 0 <= c < n_chunks - 1:
            picks |= {c, c + 1}
    if len(sizes) == 1:
        for mark_elems in (1 << 29, 1 << 28):                   # input byte 2^31 and 2^30
            if mark_elems < sizes[0]:
                picks |= {mark_elems // C - 1, mark_elems // C}
    pay_clients = list(range(clients)) if clients <= 2 * payload_clients else sorted(
        {0, 1, clients // 2, clients - 2, clients - 1} | {int(u) for u in rng.integers(0, clients, size=payload_clients)})
    one_pay = al(al(al(64 + 24) + 16) + 32)                     # payload offset of the oracle's one-chunk stream
    one_sub = al(al(64 + 24) + 16)
    g1v, mbv, mv = g1.view(clients, sess.stride), mem_before.view(clients, sess.stride), mems.view(clients, sess.stride)
    n_outlier_chunks = 0
    for c in sorted(picks):
        k = int(np.searchsorted(seg_first, c, side="right") - 1)
        start = (c - int(seg_first[k])) * C
        cnt = min(C, sizes[k] - start)
        lo = int(seg_off[k]) + start
        g_all = g1v[:, lo:lo + cnt].cpu().numpy()
        m_all = mbv[:, lo:lo + cnt].cpu().numpy()
        m_new = mv[:, lo:lo + cnt].cpu().numpy()
        wo_all = sv[:, chunk_off + 8 * c:chunk_off + 8 * c + 16].cpu().numpy().view(np.uint64).reshape(clients, 2)
        acc = np.zeros(cnt, dtype=np.float32)
        for u in range(clients):
            m = m_all[u].copy()
            r = oracle.convert(np.ascontiguousarray(g_all[u]), m, cfg["decay"], ofmts[k])
            assert same_bits(m_new[u], m), (c, u)
            n_outlier_chunks += int(r["n_saturated"] > 0)
            acc = (acc + r["ghat"]).astype(np.float32)
            st, want = oracle.encode(r["sym"], [cnt], [ocodes[k]])
            assert st == oracle.OK
            nwords = int(want[40:48].view(np.uint64)[0])
            assert int(wo_all[u, 1] - wo_all[u, 0]) == nwords, (c, u)
            if u in pay_clients:
                w0 = int(wo_all[u, 0])
                got = sv[u, pay_off + 4 * w0:pay_off + 4 * (w0 + nwords)].cpu().numpy()
                assert np.array_equal(got, want[one_pay:one_pay + 4 * nwords]), (c, u)
                got_sub = sv[u, sub_off + 32 * c:sub_off + 32 * c + 32].cpu().numpy()
                assert np.array_equal(got_sub, want[one_sub:one_sub + 32]), (c, u)
        want_avg = (acc / np.float32(clients)).astype(np.float32)
        assert same_bits(avg[lo:lo + cnt].cpu().numpy(), want_avg), c
    return dict(n_chunks=n_chunks, picks=len(picks), res=res, outlier_chunks=n_outlier_chunks)


def test_config3_full_size_sampled_chunks():
    """100 clients x 11,181,642 elements in 62 layers (4.5 GB of gradients, as much memory; the clients from the 97th
    on lie beyond byte 2^32 of both), second round with live memories, then the 100-client decode-aggregate."""
    import bench
    cfg, sizes, fmts, clients = bench.workload(3)
    assert clients == 100 and sum(sizes) == 11_181_642
    out = _full_size_sampled(cfg, list(sizes), fmts, clients, n_random=10, payload_clients=8)
    assert out["n_chunks"] == 5497


@pytest.mark.parametrize("cell", [dict(fmt=(2, 1), beta=1.0, decay=0.9), dict(fmt=(3, 0), beta=0.5, decay=0.5),
                                  dict(fmt=(4, 3), beta=2.0, decay=0.99), dict(fmt=(5, 2), beta=1.0, decay=0.9)],
                         ids=lambda c: "fmt%d%d" % c["fmt"])
def test_config4_full_size_sampled_chunks(cell):
    """The sweep's 25,600,000-element vector at full length, one cell per format (the 36 cells run at 200 k above)."""
    cfg = ci.config(4)
    assert cfg["sizes"] == (25_600_000,)
    E, M = cell["fmt"]
    c = dict(cfg, fmt=(E, M), beta=(cell["beta"],), decay=cell["decay"])
    s, inv = ci.scale_for(E, M, cell["beta"], cfg["alpha"][0])
    out = _full_size_sampled(c, list(cfg["sizes"]), [(E, M, 0, s, inv)], 1, n_random=40)
    assert out["n_chunks"] == 12500


def test_config5a_full_size_sampled_chunks():
    """1 client x 1,000,000,000 elements with 0.01 % outliers at 100x scale: 488,282 chunks, the two-level chunk
    offset scan over 120 ranges, payload bit offsets beyond 2^32."""
    import bench
    cfg, sizes, fmts, clients = bench.workload(5)
    assert clients == 1 and sizes == (1_000_000_000,)
    out = _full_size_sampled(cfg, list(sizes), fmts, 1, n_random=48)
    assert out["n_chunks"] == 488_282 and out["outlier_chunks"] > 0
    assert int(out["res"][0]["payload_bits"]) > 1 << 32


def test_config5b_full_size_sampled_chunks():
    """8 clients x 125,000,000 elements, same distribution with outliers."""
    import bench
    cfg, sizes, fmts, _ = bench.workload(5)
    part = cfg["part_b"]
    c = dict(cfg, sizes=part["sizes"])
    out = _full_size_sampled(c, list(part["sizes"]), fmts, part["clients"], n_random=24)
    assert out["n_chunks"] == 61036


def test_config2_full_size_fit_and_error_magnitude():
    """The set-up and diagnostic calls at the benchmarked size (10 clients x 11,181,642 elements in 62 layers, live
    memories after one round): every layer's fitted multiplier within one fp32 ULP of the oracle's (identical on
    nearly all), its statistics to 1e-10, and the l1 norms of every (client, layer) to 1e-12."""
    import bench
    from co3_inputs import scale_log_table
    cfg, sizes, fmts, clients = bench.workload(2)
    sess = Co3Session(sizes, fmts, clients, cfg["decay"], "cuda")
    g0 = bench.make_grads(cfg, sizes, clients, sess.stride, 0, "cuda")
    g1 = bench.make_grads(cfg, sizes, clients, sess.stride, 1, "cuda")
    mems = sess.new_client_buffer()
    sess.histogram(g0, mems, to_host=False)                     # one round: the memories are live
    norms = sess.error_magnitude(g1, mems).cpu().numpy()
    tab, beta0, dbeta = scale_log_table([tuple(cfg["fmt"])])
    stats = torch.zeros((len(sizes), 4), dtype=torch.float64, device="cuda")
    sess.fit_scales(g1, mems, torch.from_numpy(tab).cuda(), beta0, dbeta, stats_out=stats)
    torch.cuda.synchronize()
    assert sess.fit_result()[0]["status"] == co3.OK
    fm = sess.fmts_from_device()
    st_dev = stats.cpu().numpy()
    g_host = g1.cpu().numpy().reshape(clients, sess.stride)
    m_host = mems.cpu().numpy().reshape(clients, sess.stride)
    seg_off = np.concatenate([[0], np.cumsum(sizes)])
    exact = 0
    for k in range(len(sizes)):
        gk = np.ascontiguousarray(g_host[:, seg_off[k]:seg_off[k + 1]])
        mk = np.ascontiguousarray(m_host[:, seg_off[k]:seg_off[k + 1]])
        st, sc, inv, ost = oracle.fit_scale(gk, mk, cfg["decay"], tab[0], beta0, dbeta)
        assert st == oracle.OK
        d = abs(int(np.float32(fm["scale"][k]).view(np.int32)) - int(np.float32(sc).view(np.int32)))
        assert d <= 1, "layer %d" % k
        exact += d == 0
        assert fm["inv_scale"][k] == np.float32(1.0) / np.float32(fm["scale"][k])
        assert np.allclose(st_dev[k], ost, rtol=1e-10, atol=0.0)
        for u in (0, clients - 1):
            want = oracle.error_magnitude(gk[u], mk[u])
            assert np.allclose(norms[u, k], want, rtol=1e-12, atol=0.0)
    assert exact >= len(sizes) - 2
