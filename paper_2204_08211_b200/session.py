"""Convenience wrapper around the C-ABI calls for one fixed layer layout: owns the device-side
descriptor tables, the workspace and the stream buffers, and strings the entry points together
(fit codes -> encode -> decode-aggregate).  Orchestration only; all arithmetic is in libco3.so.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class Co3Session:
    def __init__(self, sizes, fmts, n_clients: int, decay: float, device="cuda"):
        """sizes: elements per layer; fmts: (exp_bits, mant_bits, flags, scale, inv_scale) per layer."""
        self.sizes = [int(n) for n in sizes]
        self.n_seg = len(self.sizes)
        self.n_elem = int(sum(self.sizes))
        self.n_clients = int(n_clients)
        self.decay = float(decay)
        self.device = torch.device(device)
        self.fmts_host = B.make_fmts(fmts)
        self.fmts = B.to_device(self.fmts_host, self.device)
        self.segs = B.to_device(B.make_segs(self.sizes), self.device)
        self.codes_host = None
        self.codes = None
        self.stride = (self.n_elem + 3) // 4 * 4                      # keeps every client's vector 16-byte aligned
        ws_bytes = B.co3_workspace_bytes(self.n_elem, self.n_seg, self.n_clients)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        self.capacity = B.co3_stream_capacity_bytes(self.n_elem, self.n_seg)
        self.streams = torch.empty(self.n_clients * self.capacity, dtype=torch.uint8, device=self.device)
        base = self.streams.data_ptr()
        self.stream_ptrs = torch.tensor([base + u * self.capacity for u in range(self.n_clients)],
                                        dtype=torch.int64, device=self.device)
        self.res_enc = torch.zeros(self.n_clients * B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        self.res_dec = torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        self.res_fit = torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        self.res_model = torch.zeros(B.RESULT_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        self.avg = torch.empty(self.n_elem, dtype=torch.float32, device=self.device)
        self.hist = torch.zeros(max(1, self.n_seg) * 256, dtype=torch.int64, device=self.device)

    # -- buffers ------------------------------------------------------------------------------
    def new_client_buffer(self, dtype=torch.float32) -> torch.Tensor:
        """Zeroed [n_clients * stride] buffer for gradients or memories."""
        return torch.zeros(self.n_clients * self.stride, dtype=dtype, device=self.device)

    def client_view(self, buf: torch.Tensor, u: int) -> torch.Tensor:
        return buf[u * self.stride:u * self.stride + self.n_elem]

    # -- multiplier fitting -------------------------------------------------------------------
    def fit_scales(self, grads: torch.Tensor, mems, log_tab: torch.Tensor, beta0: float, dbeta: float,
                   seg_tab=None, stats_out=None, stream=None) -> None:
        """Refits scale / inv_scale of every layer's format on the device from this round's gradients (and
        memories, if given): log_tab float32[n_tab][n_beta] and seg_tab int32[n_seg] (optional) are CUDA tensors.
        The host copy of the formats is stale afterwards until fmts_from_device() is called."""
        st = B.co3_fit_scale(grads, mems, self.decay, self.fmts, self.segs, self.n_seg, self.n_elem, self.n_clients,
                             self.stride, log_tab, seg_tab, log_tab.shape[0], log_tab.shape[1], beta0, dbeta,
                             stats_out, self.res_fit, self.workspace, stream)
        self._check(st, "co3_fit_scale")

    def error_magnitude(self, grads: torch.Tensor, mems: torch.Tensor, stream=None) -> torch.Tensor:
        """float64[n_clients][n_seg][2] on the device: l1 norm of each layer's gradient and memory per client."""
        out = torch.empty((self.n_clients, self.n_seg, 2), dtype=torch.float64, device=self.device)
        st = B.co3_error_magnitude(grads, mems, self.segs, self.n_seg, self.n_elem, self.n_clients, self.stride, out,
                                   self.res_fit, self.workspace, stream)
        self._check(st, "co3_error_magnitude")
        return out

    def fmts_from_device(self) -> np.ndarray:
        raw = self.fmts.cpu().numpy().tobytes()[:self.n_seg * B.FMT_DTYPE.itemsize]
        self.fmts_host = np.frombuffer(raw, dtype=B.FMT_DTYPE).copy()
        return self.fmts_host

    # -- code fitting -------------------------------------------------------------------------
    def histogram(self, grads: torch.Tensor, mems: torch.Tensor, stream=None, sym_out=None, to_host: bool = True):
        """Symbol counts per layer summed over clients for this round; `mems` is updated like a real round
        and, if `sym_out` is given, the symbols are kept for co3_encode_symbols.  The counts stay in
        self.hist on the device; to_host=False skips the copy to the host (and its synchronisation)."""
        st = B.co3_convert(grads, mems, self.decay, self.fmts, self.segs, self.n_seg, self.n_elem, self.n_clients,
                           self.stride, sym_out, self.hist, self.res_enc, self.workspace, stream)
        self._check(st, "co3_convert")
        if not to_host:
            return None
        return self.hist.cpu().numpy().astype(np.uint64).reshape(-1, 256)[:self.n_seg]

    def histogram_only(self, grads: torch.Tensor, mems: torch.Tensor, stream=None, to_host: bool = True):
        """The same counts without running the round: neither `mems` nor anything else is written."""
        st = B.co3_histogram(grads, mems, self.decay, self.fmts, self.segs, self.n_seg, self.n_elem, self.n_clients,
                             self.stride, self.hist, self.res_enc, self.workspace, stream)
        self._check(st, "co3_histogram")
        if not to_host:
            return None
        return self.hist.cpu().numpy().astype(np.uint64).reshape(-1, 256)[:self.n_seg]

    def set_codes_from_weights(self, weights: np.ndarray) -> None:
        """weights: uint64[n_seg][256] (histogram counts or model weights); one Huffman code per layer."""
        codes = np.zeros(self.n_seg, dtype=B.CODE_DTYPE)
        for k in range(self.n_seg):
            st, c = B.co3_code_build(weights[k], self.fmts_host[k:k + 1])
            self._check(st, "co3_code_build")
            codes[k] = c[0]
        self.set_codes(codes)

    def set_codes_from_histogram_device(self, stream=None) -> None:
        """One Huffman code per layer from the histogram the last histogram() call left on the device; the
        tables are built there too (the host copy of the codes is dropped)."""
        if self.codes is None:
            self.codes = torch.zeros(max(1, self.n_seg) * B.CODE_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        self.codes_host = None
        st = B.co3_code_build_device(self.hist, self.fmts, self.n_seg, self.codes, self.res_fit, stream)
        self._check(st, "co3_code_build_device")

    def set_codes_from_model_device(self, stats: torch.Tensor, stream=None) -> None:
        """One Huffman code per layer from the GenNorm model: `stats` is the float64[n_seg][4] tensor a fit_scales
        call filled (beta and alpha per layer); weights and tables are built on the device (self.hist then holds
        the model weights, not counts)."""
        st = B.co3_model_weights(self.fmts, stats, self.n_seg, self.hist, self.res_model, stream)
        self._check(st, "co3_model_weights")
        self.set_codes_from_histogram_device(stream)

    def set_codes(self, codes: np.ndarray) -> None:
        self.codes_host = codes
        self.codes = B.to_device(codes, self.device)

    # -- the two hot calls ---------------------------------------------------------------------
    def encode(self, grads: torch.Tensor, mems: torch.Tensor, stream=None) -> None:
        st = B.co3_encode(grads, mems, self.decay, self.fmts, self.codes, self.segs, self.n_seg, self.n_elem,
                          self.n_clients, self.stride, self.streams, self.capacity, self.workspace, self.res_enc,
                          stream=stream)
        self._check(st, "co3_encode")

    def encode_symbols(self, sym: torch.Tensor, stream=None) -> None:
        st = B.co3_encode_symbols(sym, self.codes, self.segs, self.n_seg, self.n_elem, self.n_clients, self.stride,
                                  self.streams, self.capacity, self.workspace, self.res_enc, stream=stream)
        self._check(st, "co3_encode_symbols")

    def decode_aggregate(self, stream=None) -> torch.Tensor:
        st = B.co3_decode_aggregate(self.stream_ptrs, self.capacity, self.n_clients, self.fmts, self.codes,
                                    self.segs, self.n_seg, self.n_elem, self.avg, self.workspace, self.res_dec,
                                    stream=stream)
        self._check(st, "co3_decode_aggregate")
        return self.avg

    def decode_aggregate_update(self, params: torch.Tensor, lr: float, want_avg: bool = False, stream=None):
        """Decode, average and apply params <- params - lr * avg in the same kernel."""
        st = B.co3_decode_aggregate_update(self.stream_ptrs, self.capacity, self.n_clients, self.fmts, self.codes,
                                           self.segs, self.n_seg, self.n_elem, lr, params,
                                           self.avg if want_avg else None, self.workspace, self.res_dec, stream=stream)
        self._check(st, "co3_decode_aggregate_update")
        return self.avg if want_avg else None

    # -- results --------------------------------------------------------------------------------
    def encode_results(self) -> np.ndarray:
        return B.read_results(self.res_enc, self.n_clients)

    def fit_result(self) -> np.ndarray:
        return B.read_results(self.res_fit, 1)

    def model_result(self) -> np.ndarray:
        return B.read_results(self.res_model, 1)

    def decode_result(self) -> np.ndarray:
        return B.read_results(self.res_dec, 1)

    def stream_bytes(self, u: int) -> np.ndarray:
        used = int(self.encode_results()[u]["container_bytes"])
        return self.streams[u * self.capacity:u * self.capacity + used].cpu().numpy()

    @staticmethod
    def _check(st: int, what: str) -> None:
        if st != B.OK:
            raise RuntimeError("%s failed: %s" % (what, B.co3_status_string(st)))
