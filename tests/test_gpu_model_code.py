"""Huffman weights from the fitted GenNorm model on the device (co3_model_weights) against the oracle's model
pmf (Sec. IV-A (ii): the code of a layer is designed for the distribution fitted to it), and the whole setup
chain without the host: moments -> shape, scale -> multiplier -> model weights -> Huffman tables -> encode.

Tolerance.  A weight is floor(p * 2^30) with p a difference of two values of the regularised incomplete gamma
function, each good to about 1e-15 on both sides (different routines): p * 2^30 agrees to ~1e-6, so a weight
differs, by one, only where p * 2^30 lies that close to an integer.  The test allows a difference of one on at
most one symbol in a thousand.  The chain test runs both sides independently from the gradients and asserts that,
on its layers, multipliers and weights come out identical, so that tables, streams and the average can be
compared bit for bit.  Needs a B200."""
import numpy as np
import pytest
import torch

import oracle
from oracle import bias
import paper_2204_08211_b200 as co3
from paper_2204_08211_b200 import binding as B
from paper_2204_08211_b200.session import Co3Session
from co3_inputs import gennorm, scale_for, scale_log_table
from harness import fmt_tuple

pytestmark = pytest.mark.gpu


def _device_weights(fmts, beta, alpha):
    n = len(fmts)
    f = B.to_device(B.make_fmts(fmts))
    stats = torch.zeros((n, 4), dtype=torch.float64, device="cuda")
    stats[:, 2] = torch.tensor(beta, dtype=torch.float64)
    stats[:, 3] = torch.tensor(alpha, dtype=torch.float64)
    w = torch.full((n * 256,), -1, dtype=torch.int64, device="cuda")
    res = torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    assert co3.co3_model_weights(f, stats, n, w, res) == co3.OK
    torch.cuda.synchronize()
    return B.read_results(res, 1)[0], w.cpu().numpy().view(np.uint64).reshape(n, 256)


def test_weights_against_the_oracle_pmf_over_formats_and_shapes():
    fmts, beta, alpha = [], [], []
    for (E, M, flush) in ((4, 3, 0), (2, 1, 0), (5, 2, 0), (3, 0, 0), (4, 3, 1), (2, 5, 0)):
        for b in (0.3, 0.5, 0.8, 1.0, 1.37, 2.0):
            for a in (1e-4, 3e-2):
                s, inv = scale_for(E, M, b, a) if (E, M) in ((4, 3), (2, 1), (5, 2), (3, 0)) else (np.float32(3.0 / a), np.float32(a / 3.0))
                fmts.append((E, M, flush, float(s), float(inv)))
                beta.append(b)
                alpha.append(a)
    res, w = _device_weights(fmts, beta, alpha)
    assert res["status"] == co3.OK
    off_by_one = 0
    for k, (E, M, flush, s, inv) in enumerate(fmts):
        want = bias.model_weights(oracle.Fmt(E, M, flush, s, inv), beta[k], alpha[k])
        d = np.abs(w[k].astype(np.int64) - want.astype(np.int64))
        assert d.max() <= 1, "layer %d: weights differ by %d" % (k, d.max())
        off_by_one += int((d == 1).sum())
        assert 2 ** 30 - 257 <= int(w[k].sum()) <= 2 ** 30 + 1
    assert off_by_one <= len(fmts) * 256 // 1000


def test_unusable_layers_are_reported():
    fmts = [fmt_tuple(4, 3, 100.0), fmt_tuple(4, 3, 100.0), (1, 3, 0, 1.0, 1.0), fmt_tuple(2, 1, 5.0)]
    res, w = _device_weights(fmts, [1.0, float("nan"), 1.0, 1.0], [1e-2, 1e-2, 1e-2, 0.0])
    assert res["status"] == co3.ERR_INVALID_ARG and res["first_bad_chunk"] == 1
    assert w[0].sum() > 0 and not w[1].any() and not w[2].any() and not w[3].any()


def test_setup_chain_on_the_device_then_encode_decode():
    """fit -> model weights -> tables -> encode -> decode on the device against the same chain through the oracle,
    each side running on its own from the gradients alone.  On these layers the two fits give identical multipliers
    and the two pmfs identical weights (asserted), so tables, streams and the average must be bit-identical."""
    sizes = [36864, 2500, 64, 147456]
    beta, alpha = [0.7, 1.1, 1.5, 0.9], [2e-3, 4e-4, 1e-2, 1e-3]
    U = 2
    g = np.stack([np.concatenate([gennorm(n, beta[k], alpha[k], 900 + 10 * u + k).numpy() for k, n in enumerate(sizes)])
                  for u in range(U)])
    tab, beta0, dbeta = scale_log_table([(4, 3)])
    sess = Co3Session(sizes, [fmt_tuple(4, 3, 1.0)] * len(sizes), U, 0.9, "cuda")
    grads, mems = sess.new_client_buffer(), sess.new_client_buffer()
    for u in range(U):
        sess.client_view(grads, u).copy_(torch.from_numpy(g[u]))
    stats = torch.zeros((len(sizes), 4), dtype=torch.float64, device="cuda")
    sess.fit_scales(grads, mems, torch.from_numpy(tab).cuda(), beta0, dbeta, stats_out=stats)
    sess.set_codes_from_model_device(stats)
    sess.encode(grads, mems)
    avg = sess.decode_aggregate().cpu().numpy()
    torch.cuda.synchronize()
    assert sess.fit_result()[0]["status"] == co3.OK and sess.model_result()[0]["status"] == co3.OK
    assert (sess.encode_results()["status"] == co3.OK).all() and sess.decode_result()[0]["status"] == co3.OK

    fm = sess.fmts_from_device()
    st_dev = stats.cpu().numpy()
    w_dev = sess.hist.cpu().numpy().view(np.uint64).reshape(-1, 256)[:len(sizes)]
    codes_dev = np.frombuffer(sess.codes.cpu().numpy().tobytes()[:len(sizes) * B.CODE_DTYPE.itemsize], dtype=B.CODE_DTYPE)
    offs = np.concatenate([[0], np.cumsum(sizes)])
    ofmts, ocodes = [], []
    for k in range(len(sizes)):
        gk = np.ascontiguousarray(g[:, offs[k]:offs[k + 1]])
        st, sc, inv, ost = oracle.fit_scale(gk, np.zeros_like(gk), 0.9, tab[0], beta0, dbeta)
        assert st == oracle.OK and fm["scale"][k] == np.float32(sc) and fm["inv_scale"][k] == np.float32(inv)
        assert np.allclose(st_dev[k], ost, rtol=1e-10, atol=0.0)
        assert abs(ost[2] - beta[k]) < 0.1 * beta[k] and abs(ost[3] - alpha[k]) < 0.15 * alpha[k]
        of = oracle.Fmt(4, 3, 0, sc, inv)
        want_w = bias.model_weights(of, float(ost[2]), float(ost[3]))
        assert np.array_equal(w_dev[k], want_w), "model weights of layer %d" % k
        code = oracle.code_build(want_w, of)
        ln, bits = oracle.code_arrays(code)
        assert np.array_equal(codes_dev["len"][k], ln) and np.array_equal(codes_dev["bits"][k].astype(np.uint32), bits)
        ofmts.append(of)
        ocodes.append(code)
    streams = []
    for u in range(U):
        sym = np.zeros(sess.n_elem, dtype=np.uint8)
        for k in range(len(sizes)):
            m = np.zeros(sizes[k], dtype=np.float32)
            sym[offs[k]:offs[k + 1]] = oracle.convert(g[u, offs[k]:offs[k + 1]], m, 0.9, ofmts[k])["sym"]
        st, s = oracle.encode(sym, sizes, ocodes)
        assert st == oracle.OK and np.array_equal(sess.stream_bytes(u), s)
        streams.append(s)
    st, want = oracle.decode_aggregate(streams, sizes, ofmts, ocodes)
    assert st == oracle.OK and np.array_equal(avg.view(np.uint32), want.view(np.uint32))
    # the model code costs little more than the entropy of the symbols it was not fitted to
    rate = float(sess.encode_results()["payload_bits"].sum()) / (U * sess.n_elem)
    assert 2.0 < rate < 8.0
