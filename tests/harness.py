"""Shared helpers of the GPU parity tests: run the same seeded inputs through the CPU oracle and
through the CUDA library (via its C ABI binding) and hand both results back for comparison."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2204_08211_b200 as co3


class Case:
    """A batch: n_clients flat gradients cut into segments with one (fmt, code) per segment."""

    def __init__(self, sizes, fmts, n_clients=1, decay=0.9, stride=None):
        self.sizes = [int(n) for n in sizes]
        self.fmts = [tuple(f) for f in fmts]            # (E, M, flags, scale, inv_scale)
        assert len(self.fmts) == len(self.sizes)
        self.n_clients = n_clients
        self.decay = decay
        self.n_elem = sum(self.sizes)
        self.stride = self.n_elem if stride is None else stride
        self.n_seg = len(self.sizes)
        self.offsets = np.concatenate([[0], np.cumsum(self.sizes)]).astype(np.int64)

    def ofmt(self, k):
        E, M, fl, s, inv = self.fmts[k]
        return oracle.Fmt(E, M, int(fl & 1), s, inv)


def fmt_tuple(E, M, scale=1.0, flush=False):
    s = np.float32(scale)
    return (E, M, 1 if flush else 0, float(s), float(np.float32(1.0) / s))


# ---------------------------------------------------------------------------------------------- oracle side
def oracle_convert(case: Case, grads, mems):
    """grads/mems: float32 arrays [n_clients][n_elem]; mems updated in place.  Returns syms, ghats, counters."""
    syms = np.zeros((case.n_clients, case.n_elem), dtype=np.uint8)
    ghats = np.zeros((case.n_clients, case.n_elem), dtype=np.float32)
    nsat = np.zeros(case.n_clients, dtype=np.uint64)
    nnf = np.zeros(case.n_clients, dtype=np.uint64)
    for u in range(case.n_clients):
        for k in range(case.n_seg):
            a, b = case.offsets[k], case.offsets[k + 1]
            m = mems[u, a:b].copy()
            r = oracle.convert(grads[u, a:b], m, case.decay, case.ofmt(k))
            mems[u, a:b] = m
            syms[u, a:b] = r["sym"]
            ghats[u, a:b] = r["ghat"]
            nsat[u] += r["n_saturated"]
            nnf[u] += r["n_nonfinite"]
    return syms, ghats, nsat, nnf


def oracle_hist(case: Case, syms):
    h = np.zeros((case.n_seg, 256), dtype=np.uint64)
    for k in range(case.n_seg):
        a, b = case.offsets[k], case.offsets[k + 1]
        for u in range(case.n_clients):
            h[k] += oracle.histogram(syms[u, a:b])
    return h


def oracle_codes(case: Case, hist):
    return [oracle.code_build(hist[k], case.ofmt(k)) for k in range(case.n_seg)]


def oracle_encode(case: Case, syms, codes):
    out = []
    for u in range(case.n_clients):
        st, s = oracle.encode(syms[u], case.sizes, codes)
        out.append((st, s))
    return out


# ---------------------------------------------------------------------------------------------- CUDA side
class Gpu:
    def __init__(self, case: Case, enc_clients=None):
        self.case = case
        self.fmts = co3.to_device(co3.make_fmts(case.fmts))
        self.segs = co3.to_device(co3.make_segs(case.sizes))
        nc = case.n_clients if enc_clients is None else enc_clients
        self.ws = torch.empty(co3.co3_workspace_bytes(case.n_elem, case.n_seg, nc) + 256, dtype=torch.uint8,
                              device="cuda")
        self.res = torch.zeros(max(1, case.n_clients) * co3.RESULT_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
        self.capacity = co3.co3_stream_capacity_bytes(case.n_elem, case.n_seg)

    def codes_dev(self, codes):
        arr = np.zeros(len(codes), dtype=co3.CODE_DTYPE)
        for k, c in enumerate(codes):
            ln, bits = oracle.code_arrays(c)
            arr[k]["len"] = ln
            arr[k]["bits"] = bits.astype(np.uint16)
        return co3.to_device(arr)

    def _buf(self, arr2d):
        c = self.case
        t = torch.zeros(c.n_clients * c.stride + 8, dtype=torch.from_numpy(arr2d[:1, :1]).dtype, device="cuda")
        for u in range(c.n_clients):
            t[u * c.stride:u * c.stride + c.n_elem] = torch.from_numpy(arr2d[u]).cuda()
        return t

    def _unbuf(self, t):
        c = self.case
        return np.stack([t[u * c.stride:u * c.stride + c.n_elem].cpu().numpy() for u in range(c.n_clients)])

    def convert(self, grads, mems, want_sym=True, want_hist=True, dither_seed=None):
        c = self.case
        g, m = self._buf(grads), self._buf(mems)
        sym = torch.full((c.n_clients * c.stride + 8,), 0xEE, dtype=torch.uint8, device="cuda") if want_sym else None
        hist = torch.full((max(1, c.n_seg) * 256,), 7, dtype=torch.int64, device="cuda") if want_hist else None
        if dither_seed is None:
            st = co3.co3_convert(g, m, c.decay, self.fmts, self.segs, c.n_seg, c.n_elem, c.n_clients, c.stride, sym,
                                 hist, self.res, self.ws)
        else:
            st = co3.co3_convert_dither(g, m, c.decay, self.fmts, self.segs, c.n_seg, c.n_elem, c.n_clients, c.stride,
                                        dither_seed, sym, hist, self.res, self.ws)
        torch.cuda.synchronize()
        res = co3.read_results(self.res, c.n_clients)
        return dict(status=st, res=res, mem=self._unbuf(m),
                    sym=self._unbuf(sym) if want_sym else None,
                    hist=hist.cpu().numpy().astype(np.uint64).reshape(-1, 256)[:c.n_seg] if want_hist else None)

    def encode(self, grads, mems, codes, capacity=None, from_sym=None, dither_seed=None):
        c = self.case
        cap = self.capacity if capacity is None else capacity
        streams = torch.full((c.n_clients * cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        codes_d = self.codes_dev(codes)
        if from_sym is None and dither_seed is not None:
            g, m = self._buf(grads), self._buf(mems)
            st = co3.co3_encode_dither(g, m, c.decay, self.fmts, codes_d, self.segs, c.n_seg, c.n_elem, c.n_clients,
                                       c.stride, dither_seed, streams, cap, self.ws, self.res)
        elif from_sym is None:
            g, m = self._buf(grads), self._buf(mems)
            st = co3.co3_encode(g, m, c.decay, self.fmts, codes_d, self.segs, c.n_seg, c.n_elem, c.n_clients, c.stride,
                                streams, cap, self.ws, self.res)
        else:
            s = self._buf(from_sym)
            m = None
            st = co3.co3_encode_symbols(s, codes_d, self.segs, c.n_seg, c.n_elem, c.n_clients, c.stride, streams, cap,
                                        self.ws, self.res)
        torch.cuda.synchronize()
        res = co3.read_results(self.res, c.n_clients)
        host = streams.cpu().numpy()
        outs = []
        for u in range(c.n_clients):
            used = int(res[u]["container_bytes"])
            outs.append(host[u * cap:u * cap + min(used, cap)].copy())
        guard_ok = bool((host[c.n_clients * cap:] == 0xA5).all())
        return dict(status=st, res=res, streams=outs, raw=host, cap=cap, guard_ok=guard_ok,
                    mem=self._unbuf(m) if m is not None else None)

    def decode(self, stream_np, codes, want_sym=True, want_val=True, stream_bytes=None):
        c = self.case
        pad = (-stream_np.size) % 16
        s = torch.from_numpy(np.concatenate([stream_np, np.zeros(pad, dtype=np.uint8)])).cuda()
        val = torch.full((c.n_elem + 8,), -77.0, dtype=torch.float32, device="cuda") if want_val else None
        sym = torch.full((c.n_elem + 8,), 0xEE, dtype=torch.uint8, device="cuda") if want_sym else None
        st = co3.co3_decode(s, s.numel() if stream_bytes is None else stream_bytes, self.fmts, self.codes_dev(codes),
                            self.segs, c.n_seg, c.n_elem, val, sym, self.ws, self.res)
        torch.cuda.synchronize()
        res = co3.read_results(self.res, 1)
        return dict(status=st, res=res, ghat=val.cpu().numpy() if want_val else None,
                    sym=sym.cpu().numpy() if want_sym else None)

    def decode_aggregate(self, streams_np, codes):
        c = self.case
        size = max(s.size for s in streams_np)
        size += (-size) % 16
        buf = torch.zeros(len(streams_np) * size, dtype=torch.uint8, device="cuda")
        for u, s in enumerate(streams_np):
            buf[u * size:u * size + s.size] = torch.from_numpy(s).cuda()
        ptrs = torch.tensor([buf.data_ptr() + u * size for u in range(len(streams_np))], dtype=torch.int64,
                            device="cuda")
        avg = torch.full((c.n_elem + 8,), -77.0, dtype=torch.float32, device="cuda")
        st = co3.co3_decode_aggregate(ptrs, size, len(streams_np), self.fmts, self.codes_dev(codes), self.segs,
                                      c.n_seg, c.n_elem, avg, self.ws, self.res)
        torch.cuda.synchronize()
        res = co3.read_results(self.res, 1)
        return dict(status=st, res=res, avg=avg.cpu().numpy())


def same_bits(a: np.ndarray, b: np.ndarray) -> bool:
    """Bit-for-bit equality of two float32 arrays (distinguishes -0 and NaN payloads)."""
    return a.shape == b.shape and np.array_equal(a.view(np.uint32), b.view(np.uint32))
