"""co3_decode_aggregate_update against the oracle (needs a B200): the model after the fused
decode + average + update must equal, bit for bit, the oracle's decode_aggregate followed by its
ps_update, for the side-by-side, the multi-batch and the single-client decoder, with ragged segments,
and over several rounds with error feedback."""
import numpy as np
import pytest
import torch

import oracle
import paper_2204_08211_b200 as co3
from co3_inputs import gennorm, scale_for
from harness import Case, Gpu, fmt_tuple, oracle_codes, oracle_convert, oracle_encode, oracle_hist, same_bits

pytestmark = pytest.mark.gpu


def _device_update(gpu, case, streams_np, codes, params_np, lr, want_avg):
    size = max(s.size for s in streams_np)
    size += (-size) % 16
    buf = torch.zeros(len(streams_np) * size, dtype=torch.uint8, device="cuda")
    for u, s in enumerate(streams_np):
        buf[u * size:u * size + s.size] = torch.from_numpy(s).cuda()
    ptrs = torch.tensor([buf.data_ptr() + u * size for u in range(len(streams_np))], dtype=torch.int64, device="cuda")
    params = torch.full((case.n_elem + 8,), 123.0, dtype=torch.float32, device="cuda")
    params[:case.n_elem] = torch.from_numpy(params_np).cuda()
    avg = torch.full((case.n_elem + 8,), -77.0, dtype=torch.float32, device="cuda") if want_avg else None
    st = co3.co3_decode_aggregate_update(ptrs, size, len(streams_np), gpu.fmts, gpu.codes_dev(codes), gpu.segs,
                                         case.n_seg, case.n_elem, lr, params, avg, gpu.ws, gpu.res)
    torch.cuda.synchronize()
    assert st == co3.OK and co3.read_results(gpu.res, 1)[0]["status"] == co3.OK
    p = params.cpu().numpy()
    assert (p[case.n_elem:] == 123.0).all(), "wrote past the model"
    if want_avg:
        a = avg.cpu().numpy()
        assert (a[case.n_elem:] == -77.0).all()
        return p[:case.n_elem], a[:case.n_elem]
    return p[:case.n_elem], None


@pytest.mark.parametrize("n_clients,want_avg", [(1, True), (2, False), (3, True), (10, True), (16, False), (17, True), (40, False)])
def test_fused_update_equals_oracle(n_clients, want_avg):
    sizes = [5000, 1, 2047, 12_289, 333]
    fmts = []
    for k, (E, M, beta) in enumerate([(4, 3, 1.0), (2, 1, 2.0), (5, 2, 0.7), (4, 3, 1.5), (3, 0, 1.0)]):
        s, inv = scale_for(E, M, beta, 1e-3)
        fmts.append((E, M, 0, s, inv))
    case = Case(sizes, fmts, n_clients=n_clients)
    rng = np.random.default_rng(100 + n_clients)
    grads = np.stack([np.concatenate([gennorm(n, 1.0, 1e-3, 7000 + 31 * u + k, "cpu").numpy() for k, n in enumerate(sizes)])
                      for u in range(n_clients)])
    syms, ghats, _, _ = oracle_convert(case, grads, np.zeros_like(grads))
    codes = oracle_codes(case, oracle_hist(case, syms))
    enc = oracle_encode(case, syms, codes)
    streams = [e[1] for e in enc]
    st, avg_want = oracle.decode_aggregate(streams, case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
    assert st == oracle.OK
    params0 = (rng.standard_normal(case.n_elem) * 0.05).astype(np.float32)
    lr = 0.0173
    want = params0.copy()
    oracle.ps_update(want, avg_want, lr)
    gpu = Gpu(case)
    got, avg_got = _device_update(gpu, case, streams, codes, params0, lr, want_avg)
    assert same_bits(got, want)
    if want_avg:
        assert same_bits(avg_got, avg_want)


def test_rounds_of_training_step_keep_model_and_memory_identical():
    """Three rounds: encode with error feedback, decode + update; model and memories follow the oracle exactly."""
    sizes = [70_000, 4099]
    fmts = []
    for E, M, beta in [(4, 3, 1.0), (4, 3, 0.6)]:
        s, inv = scale_for(E, M, beta, 1e-3)
        fmts.append((E, M, 0, s, inv))
    case = Case(sizes, fmts, n_clients=4, decay=0.9)
    gpu = Gpu(case)
    rng = np.random.default_rng(9)
    w_o = (rng.standard_normal(case.n_elem) * 0.1).astype(np.float32)
    w_g = w_o.copy()
    mem_o = np.zeros((4, case.n_elem), dtype=np.float32)
    mem_g = np.zeros((4, case.n_elem), dtype=np.float32)
    codes = None
    for rnd in range(3):
        grads = np.stack([np.concatenate([gennorm(n, 1.0, 1e-3, 900 + 17 * rnd + 5 * u + k, "cpu").numpy()
                                          for k, n in enumerate(sizes)]) for u in range(4)])
        syms, ghats, _, _ = oracle_convert(case, grads, mem_o)
        if codes is None:
            codes = oracle_codes(case, oracle_hist(case, syms))
        enc = oracle_encode(case, syms, codes)
        st, avg = oracle.decode_aggregate([e[1] for e in enc], case.sizes, [case.ofmt(k) for k in range(case.n_seg)], codes)
        assert st == oracle.OK
        oracle.ps_update(w_o, avg, 0.05)
        out = gpu.encode(grads, mem_g, codes)
        assert out["status"] == co3.OK
        mem_g = out["mem"]
        for u in range(4):
            assert np.array_equal(out["streams"][u], enc[u][1])
        w_g, _ = _device_update(gpu, case, out["streams"], codes, w_g, 0.05, False)
        assert same_bits(w_g, w_o) and same_bits(mem_g, mem_o)


def test_update_argument_checks():
    case = Case([100], [fmt_tuple(4, 3, 1.0)])
    gpu = Gpu(case)
    codes = oracle_codes(case, np.ones((1, 256), dtype=np.uint64))
    ptrs = torch.zeros(1, dtype=torch.int64, device="cuda")
    p = torch.zeros(104, dtype=torch.float32, device="cuda")
    assert co3.co3_decode_aggregate_update(ptrs, 1024, 1, gpu.fmts, gpu.codes_dev(codes), gpu.segs, 1, 100, 0.1, p[1:],
                                           None, gpu.ws, gpu.res) == co3.ERR_INVALID_ARG   # misaligned model
