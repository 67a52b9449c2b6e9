"""ctypes binding of libco3.so: argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libco3.so")

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_NO_CODEWORD, ERR_NONFINITE, ERR_CORRUPT, ERR_CUDA = range(7)
MAX_CODE_LEN, CHUNK_SYMS, SUB_SYMS = 16, 2048, 128

FMT_DTYPE = np.dtype([("exp_bits", np.uint8), ("mant_bits", np.uint8), ("flags", np.uint16),
                      ("scale", np.float32), ("inv_scale", np.float32)])
FMT_FLUSH_SUBNORMALS = 1
CODE_DTYPE = np.dtype([("len", np.uint8, (256,)), ("bits", np.uint16, (256,))])
SEG_DTYPE = np.dtype([("elem_off", np.uint64), ("n_elem", np.uint64)])
RESULT_DTYPE = np.dtype([("status", np.int32), ("first_bad_chunk", np.uint32), ("payload_bits", np.uint64),
                         ("container_bytes", np.uint64), ("n_saturated", np.uint64), ("n_nonfinite", np.uint64)])
assert FMT_DTYPE.itemsize == 12 and CODE_DTYPE.itemsize == 768 and SEG_DTYPE.itemsize == 16
assert RESULT_DTYPE.itemsize == 40

_lib = None


def library_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError("libco3.so is not built (%s): run `python -m paper_2204_08211_b200.build`; "
                           "there is no fallback path" % _LIB_PATH)
    L = C.CDLL(_LIB_PATH)
    vp, u32, u64, sz, f32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_size_t, C.c_float
    L.co3_status_string.restype = C.c_char_p
    L.co3_status_string.argtypes = [C.c_int]
    L.co3_workspace_bytes.argtypes = [u64, u32, u32, u32, C.POINTER(sz)]
    L.co3_stream_capacity_bytes.argtypes = [u64, u32, u32, C.POINTER(sz)]
    L.co3_convert.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, vp, vp, vp, vp, sz, vp]
    L.co3_histogram.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, vp, vp, vp, sz, vp]
    L.co3_convert_dither.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, u32, vp, vp, vp, vp, sz, vp]
    L.co3_histogram_dither.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, u32, vp, vp, vp, sz, vp]
    L.co3_encode_dither.argtypes = [vp, vp, f32, vp, vp, vp, u32, u64, u32, u64, u32, vp, sz, u32, vp, sz, vp, vp]
    L.co3_convert_static.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, vp, vp, vp, vp]
    L.co3_code_build.argtypes = [vp, vp, vp]
    L.co3_code_build_device.argtypes = [vp, vp, u32, vp, vp, vp]
    L.co3_fit_scale.argtypes = [vp, vp, f32, vp, vp, u32, u64, u32, u64, vp, vp, u32, u32, f32, f32, vp, vp, vp, sz, vp]
    L.co3_error_magnitude.argtypes = [vp, vp, vp, u32, u64, u32, u64, vp, vp, vp, sz, vp]
    L.co3_model_weights.argtypes = [vp, vp, u32, vp, vp, vp]
    L.co3_encode.argtypes = [vp, vp, f32, vp, vp, vp, u32, u64, u32, u64, vp, sz, u32, vp, sz, vp, vp]
    L.co3_encode_symbols.argtypes = [vp, vp, vp, u32, u64, u32, u64, vp, sz, u32, vp, sz, vp, vp]
    L.co3_decode_aggregate.argtypes = [vp, sz, u32, vp, vp, vp, u32, u64, u32, vp, vp, sz, vp, vp]
    L.co3_decode_aggregate_update.argtypes = [vp, sz, u32, vp, vp, vp, u32, u64, u32, f32, vp, vp, vp, sz, vp, vp]
    L.co3_decode.argtypes = [vp, sz, vp, vp, vp, u32, u64, u32, vp, vp, vp, sz, vp, vp]
    L.co3_profile_enable.argtypes = [C.c_int]
    L.co3_profile_read.argtypes = [vp, vp]
    for name in ("co3_histogram", "co3_convert_dither", "co3_histogram_dither", "co3_encode_dither", "co3_error_magnitude", "co3_model_weights", "co3_fit_scale", "co3_profile_enable", "co3_profile_read", "co3_convert_static", "co3_workspace_bytes", "co3_stream_capacity_bytes", "co3_convert", "co3_code_build", "co3_code_build_device", "co3_encode",
                 "co3_encode_symbols", "co3_decode_aggregate", "co3_decode_aggregate_update", "co3_decode"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _dev(t, allow_none: bool = False):
    """Device pointer of a CUDA tensor (or 0 for None)."""
    if t is None:
        if allow_none:
            return None
        raise ValueError("tensor required")
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


# ------------------------------------------------------------------------------------------------ helpers
def make_fmts(fmts) -> np.ndarray:
    """co3_fmt[n] from (exp_bits, mant_bits, flags, scale, inv_scale) tuples."""
    a = np.zeros(len(fmts), dtype=FMT_DTYPE)
    for k, f in enumerate(fmts):
        a[k] = tuple(f)
    return a


def make_segs(sizes) -> np.ndarray:
    """co3_seg[n] for contiguous segments of the given sizes."""
    a = np.zeros(len(sizes), dtype=SEG_DTYPE)
    off = 0
    for k, n in enumerate(sizes):
        a[k] = (off, int(n))
        off += int(n)
    return a


def to_device(arr: np.ndarray, device="cuda") -> torch.Tensor:
    """Raw bytes of a (structured) numpy array as a uint8 CUDA tensor (at least 16 bytes)."""
    raw = np.frombuffer(arr.tobytes(), dtype=np.uint8)
    if raw.size < 16:
        raw = np.concatenate([raw, np.zeros(16 - raw.size, dtype=np.uint8)])
    return torch.from_numpy(raw.copy()).to(device)


def read_results(res: torch.Tensor, n: int) -> np.ndarray:
    """co3_result[n] from the device buffer (synchronises)."""
    return np.frombuffer(res.cpu().numpy().tobytes()[:n * RESULT_DTYPE.itemsize], dtype=RESULT_DTYPE).copy()


# ------------------------------------------------------------------------------------------------ entry points
def co3_status_string(status: int) -> str:
    return _load().co3_status_string(int(status)).decode()


def co3_workspace_bytes(n_elem: int, n_seg: int, n_clients: int, chunk_syms: int = CHUNK_SYMS) -> int:
    out = C.c_size_t(0)
    st = _load().co3_workspace_bytes(n_elem, n_seg, n_clients, chunk_syms, C.byref(out))
    if st != OK:
        raise ValueError("co3_workspace_bytes: " + co3_status_string(st))
    return out.value


def co3_stream_capacity_bytes(n_elem: int, n_seg: int, chunk_syms: int = CHUNK_SYMS) -> int:
    out = C.c_size_t(0)
    st = _load().co3_stream_capacity_bytes(n_elem, n_seg, chunk_syms, C.byref(out))
    if st != OK:
        raise ValueError("co3_stream_capacity_bytes: " + co3_status_string(st))
    return out.value


def co3_code_build(weights: np.ndarray, fmt: np.ndarray) -> tuple[int, np.ndarray]:
    """Host call: (status, co3_code as a CODE_DTYPE scalar array of shape (1,))."""
    w = np.ascontiguousarray(weights, dtype=np.uint64)
    f = np.ascontiguousarray(fmt, dtype=FMT_DTYPE).reshape(-1)[:1].copy()
    if w.size != 256:
        raise ValueError("256 weights required")
    out = np.zeros(1, dtype=CODE_DTYPE)
    st = _load().co3_code_build(w.ctypes.data, f.ctypes.data, out.ctypes.data)
    return st, out


def co3_code_build_device(weights, fmts, n_seg, codes_out, res, stream=None) -> int:
    """Device call: weights uint64/int64[n_seg * 256], fmts and codes_out as uploaded descriptor arrays."""
    return _load().co3_code_build_device(_dev(weights), _dev(fmts), n_seg, _dev(codes_out), _dev(res), _stream(stream))


def co3_convert(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, sym_out, hist_out,
                res, workspace, stream=None) -> int:
    return _load().co3_convert(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                               n_clients, client_stride_elems, _dev(sym_out, True), _dev(hist_out, True),
                               _dev(res), _dev(workspace), workspace.numel() * workspace.element_size(),
                               _stream(stream))


def co3_histogram(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, hist_out, res,
                  workspace, stream=None) -> int:
    """Symbol counts of this round (uint64/int64[n_seg * 256]) without touching the memory or writing symbols."""
    return _load().co3_histogram(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                                 n_clients, client_stride_elems, _dev(hist_out), _dev(res), _dev(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream))


def co3_convert_dither(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, seed, sym_out,
                       hist_out, res, workspace, stream=None) -> int:
    """co3_convert with dithered (stochastic) rounding; `seed` keys the draw stream: another one every round."""
    return _load().co3_convert_dither(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                                      n_clients, client_stride_elems, int(seed), _dev(sym_out, True),
                                      _dev(hist_out, True), _dev(res), _dev(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream))


def co3_histogram_dither(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, seed, hist_out,
                         res, workspace, stream=None) -> int:
    """co3_histogram for a round that will be converted with dithered rounding under the same seed."""
    return _load().co3_histogram_dither(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                                        n_clients, client_stride_elems, int(seed), _dev(hist_out), _dev(res),
                                        _dev(workspace), workspace.numel() * workspace.element_size(),
                                        _stream(stream))


def co3_encode_dither(grad, mem, decay, fmts, codes, segs, n_seg, n_elem, n_clients, client_stride_elems, seed,
                      streams_out, stream_capacity, workspace, res, chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    """co3_encode with dithered (stochastic) rounding."""
    return _load().co3_encode_dither(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(codes), _dev(segs), n_seg,
                                     n_elem, n_clients, client_stride_elems, int(seed), _dev(streams_out),
                                     stream_capacity, chunk_syms, _dev(workspace),
                                     workspace.numel() * workspace.element_size(), _dev(res), _stream(stream))


STATIC_SCRATCH_BYTES = 2 << 20


def co3_convert_static(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, sym_out, hist_out,
                       res, stream=None) -> int:
    """co3_convert on the library's built-in scratch array: no workspace tensor, nothing is allocated.
    For hosts that may not allocate device memory where they call this; layouts needing more than
    STATIC_SCRATCH_BYTES of workspace return ERR_CAPACITY.  Calls on one device share the array: order them."""
    return _load().co3_convert_static(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                                      n_clients, client_stride_elems, _dev(sym_out, True), _dev(hist_out, True),
                                      _dev(res), _stream(stream))


def co3_fit_scale(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, log_tab, seg_tab,
                  n_tab, n_beta, beta0, dbeta, stats_out, res, workspace, stream=None) -> int:
    """Writes scale / inv_scale of every layer's co3_fmt on the device; mem, seg_tab, stats_out may be None."""
    return _load().co3_fit_scale(_dev(grad), _dev(mem, True), float(decay), _dev(fmts), _dev(segs), n_seg, n_elem,
                                 n_clients, client_stride_elems, _dev(log_tab), _dev(seg_tab, True), n_tab, n_beta,
                                 float(beta0), float(dbeta), _dev(stats_out, True), _dev(res), _dev(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream))


def co3_error_magnitude(grad, mem, segs, n_seg, n_elem, n_clients, client_stride_elems, norms_out, res, workspace,
                        stream=None) -> int:
    """norms_out float64[n_clients * n_seg * 2]: l1 norms of gradient and memory per client and layer."""
    return _load().co3_error_magnitude(_dev(grad), _dev(mem), _dev(segs), n_seg, n_elem, n_clients, client_stride_elems,
                                       _dev(norms_out), _dev(res), _dev(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream))


def co3_model_weights(fmts, stats, n_seg, weights_out, res, stream=None) -> int:
    """weights_out int64/uint64[n_seg * 256] from the formats and the (beta, alpha) columns of co3_fit_scale's stats."""
    return _load().co3_model_weights(_dev(fmts), _dev(stats), n_seg, _dev(weights_out), _dev(res), _stream(stream))


def co3_encode(grad, mem, decay, fmts, codes, segs, n_seg, n_elem, n_clients, client_stride_elems, streams_out,
               stream_capacity, workspace, res, chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    return _load().co3_encode(_dev(grad), _dev(mem), float(decay), _dev(fmts), _dev(codes), _dev(segs), n_seg,
                              n_elem, n_clients, client_stride_elems, _dev(streams_out), stream_capacity, chunk_syms,
                              _dev(workspace), workspace.numel() * workspace.element_size(), _dev(res),
                              _stream(stream))


def co3_encode_symbols(sym, codes, segs, n_seg, n_elem, n_clients, client_stride_elems, streams_out,
                       stream_capacity, workspace, res, chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    return _load().co3_encode_symbols(_dev(sym), _dev(codes), _dev(segs), n_seg, n_elem, n_clients,
                                      client_stride_elems, _dev(streams_out), stream_capacity, chunk_syms,
                                      _dev(workspace), workspace.numel() * workspace.element_size(), _dev(res),
                                      _stream(stream))


def co3_decode_aggregate(stream_ptrs, stream_bytes, n_clients, fmts, codes, segs, n_seg, n_elem, avg_out, workspace,
                         res, chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    """stream_ptrs: int64 CUDA tensor holding the n_clients device addresses of the streams."""
    return _load().co3_decode_aggregate(_dev(stream_ptrs), stream_bytes, n_clients, _dev(fmts), _dev(codes),
                                        _dev(segs), n_seg, n_elem, chunk_syms, _dev(avg_out), _dev(workspace),
                                        workspace.numel() * workspace.element_size(), _dev(res), _stream(stream))


def co3_decode_aggregate_update(stream_ptrs, stream_bytes, n_clients, fmts, codes, segs, n_seg, n_elem, lr, params,
                                avg_out, workspace, res, chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    """co3_decode_aggregate with params <- params - lr * avg folded in; avg_out may be None."""
    return _load().co3_decode_aggregate_update(_dev(stream_ptrs), stream_bytes, n_clients, _dev(fmts), _dev(codes),
                                               _dev(segs), n_seg, n_elem, chunk_syms, float(lr), _dev(params),
                                               _dev(avg_out, True), _dev(workspace),
                                               workspace.numel() * workspace.element_size(), _dev(res), _stream(stream))


def co3_decode(stream_in, stream_bytes, fmts, codes, segs, n_seg, n_elem, ghat_out, sym_out, workspace, res,
               chunk_syms: int = CHUNK_SYMS, stream=None) -> int:
    return _load().co3_decode(_dev(stream_in), stream_bytes, _dev(fmts), _dev(codes), _dev(segs), n_seg, n_elem,
                              chunk_syms, _dev(ghat_out, True), _dev(sym_out, True), _dev(workspace),
                              workspace.numel() * workspace.element_size(), _dev(res), _stream(stream))


KERNEL_NAMES = ("prepare", "convert", "pack", "scan", "compact", "code_build", "decode", "fit", "clear")


def co3_profile_enable(on: bool) -> int:
    return _load().co3_profile_enable(1 if on else 0)


def co3_profile_read() -> dict:
    """{kernel name: (launches, total ms)} since profiling was enabled or last read (synchronises)."""
    ms = np.zeros(len(KERNEL_NAMES), dtype=np.float64)
    n = np.zeros(len(KERNEL_NAMES), dtype=np.uint32)
    st = _load().co3_profile_read(ms.ctypes.data, n.ctypes.data)
    if st != OK:
        raise RuntimeError("co3_profile_read: " + co3_status_string(st))
    return {k: (int(n[i]), float(ms[i])) for i, k in enumerate(KERNEL_NAMES)}
