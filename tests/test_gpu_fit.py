"""Per-layer fit of the converter's multiplier on the device (co3_fit_scale) against the oracle's fit
(Sec. III: zero-mean GenNorm model, its kurtosis and variance; Sec. IV-A (i): the multiplier that minimises the
conversion error, tabulated per shape).

Tolerance.  Both sides add fp64 squares and fourth powers of the same fp32 values, in different orders, and
evaluate the same formulas with different lgamma/exp routines: the moments agree to a few 1e-13 relative (N up
to 1e7 terms, error growth ~ sqrt(N) * 2^-53), the fitted shape and the multiplier to ~1e-11 before the
multiplier is rounded to fp32.  So the fp32 multiplier is identical unless the fp64 value lies within 1e-11 of
a rounding boundary: the tests allow one fp32 ULP per layer and demand identity for nearly all layers; the
stored reciprocal must be fl32(1 / scale) of the scale the device wrote.  Needs a B200."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from paper_2204_08211_b200 import binding as B
from paper_2204_08211_b200.session import Co3Session
from co3_inputs import gennorm, layer_params, scale_log_table
from harness import fmt_tuple

pytestmark = pytest.mark.gpu

FORMATS = [(4, 3), (2, 1), (5, 2), (3, 0)]


def _ulp_apart(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    return np.abs(a.astype(np.float32).view(np.int32).astype(np.int64) - b.astype(np.float32).view(np.int32).astype(np.int64))


def _run(sizes, g_host, m_host, decay, seg_tab, n_clients, poison_fmt=False):
    """Device fit and oracle fit of the same buffers.  g_host/m_host: float32 [n_clients][n_elem] (m may be None)."""
    tab, beta0, dbeta = scale_log_table(FORMATS)
    fmts = [fmt_tuple(*FORMATS[t], 1.0) for t in seg_tab]
    if poison_fmt:  # whatever multiplier was there before must not matter (not even an invalid one)
        fmts = [(E, M, fl, float("nan"), -1.0) for (E, M, fl, _, _) in fmts]
    sess = Co3Session(sizes, fmts, n_clients, decay, "cuda")
    grads = sess.new_client_buffer()
    mems = sess.new_client_buffer() if m_host is not None else None
    for u in range(n_clients):
        sess.client_view(grads, u).copy_(torch.from_numpy(g_host[u]))
        if mems is not None:
            sess.client_view(mems, u).copy_(torch.from_numpy(m_host[u]))
    g_before = grads.clone()
    d_tab = torch.from_numpy(tab).cuda()
    d_seg_tab = torch.tensor(seg_tab, dtype=torch.int32, device="cuda")
    stats = torch.full((len(sizes), 4), -1.0, dtype=torch.float64, device="cuda")
    sess.fit_scales(grads, mems, d_tab, beta0, dbeta, seg_tab=d_seg_tab, stats_out=stats)
    torch.cuda.synchronize()
    assert torch.equal(grads.view(torch.int32), g_before.view(torch.int32))     # inputs are read only
    got = sess.fmts_from_device().copy()
    res = sess.fit_result()[0]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    want = []
    for k, n in enumerate(sizes):
        g = np.ascontiguousarray(g_host[:, offs[k]:offs[k + 1]])
        m = None if m_host is None else np.ascontiguousarray(m_host[:, offs[k]:offs[k + 1]])
        want.append(oracle.fit_scale(g, m, decay, tab[seg_tab[k]], beta0, dbeta))
    return got, stats.cpu().numpy(), res, want, fmts


def _compare(got, stats, want, min_exact):
    exact = 0
    for k, (st, sc, inv, ost) in enumerate(want):
        assert st == oracle.OK
        d = int(_ulp_apart(np.array([got["scale"][k]]), np.array([sc]))[0])
        assert d <= 1, "layer %d: multiplier %r vs %r" % (k, got["scale"][k], sc)
        exact += d == 0
        assert got["inv_scale"][k] == np.float32(1.0) / np.float32(got["scale"][k])
        assert np.allclose(stats[k], ost, rtol=1e-10, atol=0.0), "layer %d statistics" % k
    assert exact >= min_exact, "%d of %d multipliers identical" % (exact, len(want))


def test_layered_gradients_several_clients_with_memory():
    # ragged layers (not multiples of the chunk, odd offsets), four formats with their own tables, three clients
    sizes = [9408, 64, 36864, 10, 2048, 2049, 4095, 147456, 513, 70001]
    beta, alpha = layer_params(len(sizes), seed=5, beta_range=(0.5, 1.8))
    seg_tab = [k % len(FORMATS) for k in range(len(sizes))]
    U = 3
    g = np.stack([np.concatenate([gennorm(n, beta[k], alpha[k], 100 * u + k).numpy() for k, n in enumerate(sizes)])
                  for u in range(U)])
    m = np.stack([np.concatenate([gennorm(n, 1.0, 0.3 * alpha[k], 7000 + 100 * u + k).numpy() for k, n in enumerate(sizes)])
                  for u in range(U)])
    got, stats, res, want, fmts = _run(sizes, g, m, 0.9, seg_tab, U, poison_fmt=True)
    assert res["status"] == co3.OK
    _compare(got, stats, want, min_exact=len(sizes) - 1)
    # the other fields of the formats are untouched
    assert [int(e) for e in got["exp_bits"]] == [f[0] for f in fmts]
    assert [int(e) for e in got["mant_bits"]] == [f[1] for f in fmts]


def test_without_memory_and_one_client_long_layer():
    sizes = [3_000_001, 777]
    g = np.concatenate([gennorm(sizes[0], 0.8, 1e-3, 1, outlier_frac=1e-4, outlier_mult=100.0).numpy(),
                        gennorm(sizes[1], 2.0, 5e-2, 2).numpy()])[None, :]
    got, stats, res, want, _ = _run(sizes, g, None, 0.9, [0, 0], 1)
    assert res["status"] == co3.OK
    _compare(got, stats, want, min_exact=1)


def test_shapes_outside_the_table_take_its_ends():
    # +-a only: kurtosis 1, lighter tails than any tabulated shape -> the table's last node (closed form on the
    # oracle side: alpha = a * sqrt(Gamma(1/b) / Gamma(3/b)) at that node); a few huge entries among zeros: its first
    a = 0.25
    two_point = np.tile(np.array([a, -a], dtype=np.float32), 3000)
    spikes = np.zeros(50000, dtype=np.float32)
    spikes[::5000] = 3.0
    g = np.concatenate([two_point, spikes])[None, :]
    got, stats, res, want, _ = _run([two_point.size, spikes.size], g, None, 0.0, [0, 1], 1)
    assert res["status"] == co3.OK
    _compare(got, stats, want, min_exact=2)
    tab, beta0, dbeta = scale_log_table(FORMATS)
    assert stats[0][1] == 1.0 and stats[0][2] == np.float32(beta0) + np.float64(np.float32(dbeta)) * (tab.shape[1] - 1)
    assert stats[1][2] == np.float64(np.float32(beta0))


def test_layers_without_a_fit_are_reported_and_left_alone():
    sizes = [5000, 4096, 300, 2048]
    g = np.concatenate([gennorm(5000, 1.0, 1e-3, 3).numpy(), np.zeros(4096, dtype=np.float32),
                        gennorm(300, 1.0, 1e-3, 4).numpy(), gennorm(2048, 1.0, 1e-3, 5).numpy()])[None, :].copy()
    g[0, 5000 + 4096 + 17] = np.nan
    got, stats, res, want, fmts = _run(sizes, g, None, 0.0, [0, 0, 0, 0], 1)
    assert res["status"] == co3.ERR_INVALID_ARG and res["first_bad_chunk"] == 1
    assert want[1][0] != oracle.OK and want[2][0] != oracle.OK
    for k in (1, 2):       # untouched: still what the session uploaded
        assert got["scale"][k] == np.float32(fmts[k][3]) and got["inv_scale"][k] == np.float32(fmts[k][4])
        assert (stats[k] == -1.0).all()
    for k in (0, 3):
        assert want[k][0] == oracle.OK and _ulp_apart(np.array([got["scale"][k]]), np.array([want[k][1]]))[0] <= 1


def test_fitted_formats_drive_the_conversion():
    """Fit then convert, each side on its own: the device converts with the formats its fit left on the device, the
    oracle with the multipliers of the oracle's fit.  On these layers the two fits give identical fp32 multipliers
    (asserted), so symbols and memories must be bit-identical."""
    sizes = [36864, 2500, 64]
    beta, alpha = [0.7, 1.1, 1.5], [2e-3, 4e-4, 1e-2]
    g = np.concatenate([gennorm(n, beta[k], alpha[k], 50 + k).numpy() for k, n in enumerate(sizes)])[None, :]
    tab, beta0, dbeta = scale_log_table([(4, 3)])
    sess = Co3Session(sizes, [fmt_tuple(4, 3, 1.0)] * 3, 1, 0.9, "cuda")
    grads, mems = sess.new_client_buffer(), sess.new_client_buffer()
    sess.client_view(grads, 0).copy_(torch.from_numpy(g[0]))
    sess.fit_scales(grads, mems, torch.from_numpy(tab).cuda(), beta0, dbeta)
    sym = torch.zeros(sess.stride, dtype=torch.uint8, device="cuda")
    sess.histogram(grads, mems, sym_out=sym)
    torch.cuda.synchronize()
    fm = sess.fmts_from_device()
    offs = np.concatenate([[0], np.cumsum(sizes)])
    for k in range(3):
        gk = np.ascontiguousarray(g[0, offs[k]:offs[k + 1]])
        st, sc, inv, _ = oracle.fit_scale(gk, np.zeros_like(gk), 0.9, tab[0], beta0, dbeta)
        assert st == oracle.OK and fm["scale"][k] == np.float32(sc) and fm["inv_scale"][k] == np.float32(inv)
        m = np.zeros(sizes[k], dtype=np.float32)
        r = oracle.convert(gk, m, 0.9, oracle.Fmt(4, 3, 0, sc, inv))
        assert np.array_equal(sym[offs[k]:offs[k + 1]].cpu().numpy(), r["sym"])
        assert np.array_equal(sess.client_view(mems, 0)[offs[k]:offs[k + 1]].cpu().numpy().view(np.uint32), m.view(np.uint32))
        assert r["n_saturated"] < 0.001 * sizes[k]      # the fitted multiplier keeps the layer inside the format


def test_argument_checks():
    sess = Co3Session([4096], [fmt_tuple(4, 3, 1.0)], 1, 0.9, "cuda")
    tab, beta0, dbeta = scale_log_table([(4, 3)])
    d_tab = torch.from_numpy(tab).cuda()
    g = sess.new_client_buffer()
    args = dict(n_seg=1, n_elem=4096, n_clients=1, client_stride_elems=sess.stride, seg_tab=None, n_tab=1,
                n_beta=tab.shape[1], beta0=beta0, dbeta=dbeta, stats_out=None, res=sess.res_fit, workspace=sess.workspace)
    call = lambda **kw: co3.co3_fit_scale(g, None, 0.9, sess.fmts, sess.segs, log_tab=d_tab, **{**args, **kw})
    assert call() == co3.OK
    assert call(n_beta=1) == co3.ERR_INVALID_ARG
    assert call(dbeta=0.0) == co3.ERR_INVALID_ARG
    assert call(n_clients=0) == co3.ERR_INVALID_ARG
    assert call(workspace=sess.workspace[:4096]) == co3.ERR_CAPACITY
    torch.cuda.synchronize()


def test_inconsistent_segment_table_is_refused_on_the_device():
    """A segment table that does not tile the vector is found by the layout check on the device: the status says
    so, no format is written, and the error-magnitude call on the same table reports it too (output untouched)."""
    sess = Co3Session([4096, 1000], [fmt_tuple(4, 3, 2.0)] * 2, 1, 0.9, "cuda")
    bad = B.make_segs([4096, 1000])
    bad[1]["elem_off"] = 4000                       # overlaps the first layer
    segs = B.to_device(bad)
    tab, beta0, dbeta = scale_log_table([(4, 3)])
    g = sess.new_client_buffer()
    g.normal_(0.0, 1e-3, generator=torch.Generator(device="cuda").manual_seed(1))
    st = co3.co3_fit_scale(g, None, 0.9, sess.fmts, segs, 2, sess.n_elem, 1, sess.stride, torch.from_numpy(tab).cuda(),
                           None, 1, tab.shape[1], beta0, dbeta, None, sess.res_fit, sess.workspace)
    assert st == co3.OK
    torch.cuda.synchronize()
    assert sess.fit_result()[0]["status"] == co3.ERR_INVALID_ARG
    fm = sess.fmts_from_device()
    assert (fm["scale"] == np.float32(2.0)).all() and (fm["inv_scale"] == np.float32(0.5)).all()
    norms = torch.full((1, 2, 2), -7.0, dtype=torch.float64, device="cuda")
    st = co3.co3_error_magnitude(g, g, segs, 2, sess.n_elem, 1, sess.stride, norms, sess.res_fit, sess.workspace)
    assert st == co3.OK
    torch.cuda.synchronize()
    assert sess.fit_result()[0]["status"] == co3.ERR_INVALID_ARG and (norms == -7.0).all()
