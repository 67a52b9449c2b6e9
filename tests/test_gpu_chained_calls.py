"""Several rounds of calls enqueued on one stream without a host synchronisation in between (needs a B200).

Every kernel of the library is launched so that its launch may overlap the kernel before it and waits on the device
for that kernel's results; a call also clears and rebuilds the state in the workspace that the call before it used.
Four rounds of dry histogram, encode and decode-aggregate-update are queued in one go here and only then compared,
round by round, with the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, fmt_tuple, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits
from paper_2204_08211_b200.session import Co3Session

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_clients", [1, 3, 18])
def test_rounds_queued_back_to_back(n_clients):
    sizes = [70_000, 10, 2048, 0, 4099, 150_000, 63]
    fmts = []
    for k in range(len(sizes)):
        E, M = [(4, 3), (2, 1), (5, 2), (3, 0)][k % 4]
        fmts.append(fmt_tuple(E, M, scale_for(E, M, 1.0, 1e-3)[0], flush=(k == 4)))
    case = Case(sizes, fmts, n_clients=n_clients, decay=0.9)
    rounds, lr = 4, np.float32(0.05)
    sess = Co3Session(sizes, fmts, n_clients, 0.9, "cuda")
    g_np = [np.stack([gennorm(case.n_elem, 1.0, 1e-3, seed=900 + 50 * r + u).numpy() for u in range(n_clients)])
            for r in range(rounds)]

    # the oracle's rounds (and the code, from its first round's symbols)
    mem_o = np.zeros((n_clients, case.n_elem), dtype=np.float32)
    w_o = gennorm(case.n_elem, 2.0, 0.1, seed=7).numpy().astype(np.float32)
    w0 = w_o.copy()
    codes, want_streams, want_avg, want_hist = None, [], [], []
    for r in range(rounds):
        syms, _, _, _ = oracle_convert(case, g_np[r], mem_o)
        want_hist.append(oracle_hist(case, syms))
        if codes is None:
            codes = oracle_codes(case, want_hist[0])
        enc = oracle_encode(case, syms, codes)
        want_streams.append([s for _, s in enc])
        st, avg = oracle.decode_aggregate(want_streams[-1], case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
        assert st == oracle.OK
        want_avg.append(avg.copy())
        oracle.ps_update(w_o, avg, float(lr))
    ln = np.stack([oracle.code_arrays(c)[0] for c in codes])
    bits = np.stack([oracle.code_arrays(c)[1] for c in codes])
    from paper_2204_08211_b200.binding import CODE_DTYPE
    code_np = np.zeros(case.n_seg, dtype=CODE_DTYPE)
    code_np["len"], code_np["bits"] = ln, bits
    sess.set_codes(code_np)

    # the same rounds on the device, all queued before anything is looked at
    grads = []
    for r in range(rounds):
        buf = sess.new_client_buffer()
        for u in range(n_clients):
            sess.client_view(buf, u)[:case.n_elem] = torch.from_numpy(g_np[r][u])
        grads.append(buf)
    mems = sess.new_client_buffer()
    params = torch.from_numpy(w0).cuda()
    got_avg = torch.zeros((rounds, case.n_elem), dtype=torch.float32, device="cuda")
    got_hist = torch.zeros((rounds, case.n_seg * 256), dtype=torch.int64, device="cuda")
    got_streams = torch.zeros((rounds, sess.streams.numel()), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    for r in range(rounds):
        sess.histogram_only(grads[r], mems, to_host=False)
        got_hist[r].copy_(sess.hist.view(-1)[:case.n_seg * 256])
        sess.encode(grads[r], mems)
        got_streams[r].copy_(sess.streams)
        avg = sess.decode_aggregate_update(params, float(lr), want_avg=True)
        got_avg[r].copy_(avg[:case.n_elem])
    torch.cuda.synchronize()

    assert (sess.encode_results()["status"] == co3.OK).all() and sess.decode_result()["status"][0] == co3.OK
    for r in range(rounds):
        assert np.array_equal(got_hist[r].cpu().numpy().astype(np.uint64).reshape(-1, 256), want_hist[r])
        assert same_bits(got_avg[r].cpu().numpy(), want_avg[r])
        for u in range(n_clients):
            want = want_streams[r][u]
            got = got_streams[r][u * sess.capacity:u * sess.capacity + want.size].cpu().numpy()
            assert np.array_equal(got, want)
    for u in range(n_clients):
        assert same_bits(sess.client_view(mems, u)[:case.n_elem].cpu().numpy(), mem_o[u])
    assert same_bits(params.cpu().numpy(), w_o)
