"""l1 norms of gradient and memory per client and layer on the device (co3_error_magnitude) against the oracle
(Sec. VI, "Error magnitude").  Both sides add the same fp64 terms in different orders: relative agreement to
1e-12 (n up to a few million terms, growth ~ sqrt(n) * 2^-53), identity where the sums are exact.  Needs a B200."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from paper_2204_08211_b200.session import Co3Session
from co3_inputs import gennorm
from harness import fmt_tuple

pytestmark = pytest.mark.gpu


def _both(sizes, g, m):
    U = g.shape[0]
    sess = Co3Session(sizes, [fmt_tuple(4, 3, 1.0)] * len(sizes), U, 0.9, "cuda")
    grads, mems = sess.new_client_buffer(), sess.new_client_buffer()
    for u in range(U):
        sess.client_view(grads, u).copy_(torch.from_numpy(g[u]))
        sess.client_view(mems, u).copy_(torch.from_numpy(m[u]))
    got = sess.error_magnitude(grads, mems).cpu().numpy()
    assert sess.fit_result()[0]["status"] == co3.OK
    offs = np.concatenate([[0], np.cumsum(sizes)])
    want = np.array([[oracle.error_magnitude(g[u, offs[k]:offs[k + 1]], m[u, offs[k]:offs[k + 1]])
                      for k in range(len(sizes))] for u in range(U)])
    return got, want, sess, grads, mems


def test_layered_batches_ragged_layers():
    sizes = [9408, 64, 1, 2048, 2049, 300001, 4095, 10]
    U = 3
    g = np.stack([np.concatenate([gennorm(n, 0.9, 1e-3 * (k + 1), 10 * u + k).numpy() for k, n in enumerate(sizes)]) for u in range(U)])
    m = np.stack([np.concatenate([gennorm(n, 1.3, 2e-4 * (k + 1), 500 + 10 * u + k).numpy() for k, n in enumerate(sizes)]) for u in range(U)])
    got, want, *_ = _both(sizes, g, m)
    assert got.shape == want.shape == (U, len(sizes), 2)
    assert np.allclose(got, want, rtol=1e-12, atol=0.0)
    assert not np.allclose(got[..., 0], want[..., 1], rtol=1e-3)       # the two norms are not swapped


def test_exact_sums_long_layer_and_nonfinite_values():
    # magnitudes that are multiples of 2^-10 below 2^10: every partial sum is exact, so any order gives the same bits
    rng = np.random.default_rng(5)
    sizes = [3_000_000, 5000, 4096]
    n = sum(sizes)
    g = (rng.integers(-2 ** 20, 2 ** 20, size=(1, n)) / 1024.0).astype(np.float32)
    m = (rng.integers(-2 ** 12, 2 ** 12, size=(1, n)) / 1024.0).astype(np.float32)
    m[0, 3_000_000 + 77] = np.nan
    g[0, 3_005_000 + 5] = -np.inf
    got, want, *_ = _both(sizes, g, m)
    assert np.array_equal(got[0, 0], want[0, 0]) and got[0, 0, 0] == np.abs(g[0, :3_000_000].astype(np.float64)).sum()
    assert got[0, 1, 0] == want[0, 1, 0] and math.isnan(got[0, 1, 1]) and math.isnan(want[0, 1, 1])
    assert got[0, 2, 0] == np.inf and got[0, 2, 1] == want[0, 2, 1]


def test_memory_against_gradient_over_rounds():
    """The figure of Sec. VI: with error feedback the memory settles at a fraction of the gradient's size; device
    rounds (convert with memory) and oracle rounds give the same norms round after round."""
    from co3_inputs import scale_for
    sizes = [50000, 3000]
    beta, alpha = [1.0, 0.8], [1e-3, 2e-3]
    fmts = [(2, 1, 0) + scale_for(2, 1, beta[k], alpha[k]) for k in range(2)]
    sess = Co3Session(sizes, fmts, 1, 0.9, "cuda")
    grads, mems = sess.new_client_buffer(), sess.new_client_buffer()
    m_host = np.zeros(sess.n_elem, dtype=np.float32)
    offs = [0, sizes[0], sum(sizes)]
    for rnd in range(4):
        g = np.concatenate([gennorm(n, beta[k], alpha[k], 100 * rnd + k).numpy() for k, n in enumerate(sizes)])
        sess.client_view(grads, 0).copy_(torch.from_numpy(g))
        sess.histogram(grads, mems, to_host=False)
        got = sess.error_magnitude(grads, mems).cpu().numpy()[0]
        for k in range(2):
            mk = m_host[offs[k]:offs[k + 1]].copy()
            oracle.convert(g[offs[k]:offs[k + 1]], mk, 0.9, oracle.Fmt(2, 1, 0, fmts[k][3], fmts[k][4]))
            m_host[offs[k]:offs[k + 1]] = mk
            want = oracle.error_magnitude(g[offs[k]:offs[k + 1]], mk)
            assert np.allclose(got[k], want, rtol=1e-12, atol=0.0)
            assert 0.05 * want[0] < want[1] < 1.5 * want[0]
