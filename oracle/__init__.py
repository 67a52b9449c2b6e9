"""CPU oracle for the CO3 uplink pipeline — TEST INFRASTRUCTURE, not a product path.

Thin ctypes access to ``co3_oracle.c`` (plain C, single thread, written from the paper).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA library and its Python binding never do, and the two share no code.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "co3_oracle.c")
_LIB = os.path.join(_HERE, "libco3_oracle.so")

OK, ERR_ARG, ERR_CAPACITY, ERR_NO_CODEWORD, ERR_CORRUPT = 0, 1, 2, 3, 5
MAX_CODE_LEN = 16


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction of a*b+c, no fast math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
             "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Fmt(C.Structure):
    _fields_ = [("exp_bits", C.c_int32), ("mant_bits", C.c_int32), ("flush_subnormals", C.c_int32),
                ("scale", C.c_float), ("inv_scale", C.c_float)]


class Code(C.Structure):
    _fields_ = [("len", C.c_uint8 * 256), ("bits", C.c_uint32 * 256)]


def make_fmt(exp_bits: int, mant_bits: int, scale: float = 1.0, flush_subnormals: bool = False) -> Fmt:
    s = np.float32(scale)
    inv = np.float32(1.0) / s
    return Fmt(exp_bits, mant_bits, int(flush_subnormals), float(s), float(inv))


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.co3o_level.restype = C.c_double
        L.co3o_level.argtypes = [C.POINTER(Fmt), C.c_uint32]
        L.co3o_max_code.restype = C.c_uint32
        L.co3o_max_code.argtypes = [C.POINTER(Fmt)]
        L.co3o_symbol_valid.restype = C.c_int
        L.co3o_symbol_valid.argtypes = [C.POINTER(Fmt), C.c_uint32]
        L.co3o_symbol_value.restype = C.c_float
        L.co3o_symbol_value.argtypes = [C.POINTER(Fmt), C.c_uint32]
        L.co3o_fmt_ok.restype = C.c_int
        L.co3o_fmt_ok.argtypes = [C.POINTER(Fmt)]
        L.co3o_convert.restype = C.c_int
        L.co3o_convert.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.POINTER(Fmt), C.c_uint64,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.co3o_histogram.restype = None
        L.co3o_philox4x32_10.restype = None
        L.co3o_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.co3o_dither_draws.restype = None
        L.co3o_dither_draws.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64, C.c_void_p]
        L.co3o_convert_dithered.restype = C.c_int
        L.co3o_convert_dithered.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.POINTER(Fmt), C.c_uint64, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.co3o_histogram.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        L.co3o_code_build.restype = C.c_int
        L.co3o_code_build.argtypes = [C.c_void_p, C.POINTER(Fmt), C.POINTER(Code)]
        L.co3o_stream_capacity_bytes.restype = C.c_int
        L.co3o_stream_capacity_bytes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32,
                                                 C.POINTER(C.c_uint64)]
        L.co3o_encode.restype = C.c_int
        L.co3o_encode.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32,
                                  C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64)]
        L.co3o_decode.restype = C.c_int
        L.co3o_decode.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32,
                                  C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p]
        L.co3o_decode_aggregate.restype = C.c_int
        L.co3o_decode_aggregate.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p,
                                            C.c_void_p]
        L.co3o_gennorm_kurtosis.restype = C.c_double
        L.co3o_gennorm_kurtosis.argtypes = [C.c_double]
        L.co3o_gennorm_shape_from_kurtosis.restype = C.c_double
        L.co3o_gennorm_shape_from_kurtosis.argtypes = [C.c_double, C.c_double, C.c_double]
        L.co3o_fit_scale.restype = C.c_int
        L.co3o_fit_scale.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_uint64, C.c_uint32, C.c_uint64,
                                     C.c_void_p, C.c_uint32, C.c_float, C.c_float,
                                     C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_void_p]
        L.co3o_error_magnitude.restype = None
        L.co3o_error_magnitude.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        L.co3o_ps_update.restype = None
        L.co3o_ps_update.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_uint64]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ------------------------------------------------------------------------------------------ levels
def level(fmt: Fmt, code: int) -> float:
    return float(lib().co3o_level(C.byref(fmt), code))


def levels(fmt: Fmt):
    """(codes, magnitudes) of every magnitude code the converter can produce, in increasing order."""
    n = 1 << (fmt.exp_bits + fmt.mant_bits)
    cs, ls = [], []
    for c in range(n):
        lv = level(fmt, c)
        if lv >= 0.0:
            cs.append(c)
            ls.append(lv)
    return np.array(cs, dtype=np.uint32), np.array(ls, dtype=np.float64)


def max_code(fmt: Fmt) -> int:
    return int(lib().co3o_max_code(C.byref(fmt)))


def symbol_valid(fmt: Fmt, sym: int) -> bool:
    return bool(lib().co3o_symbol_valid(C.byref(fmt), sym))


def symbol_value(fmt: Fmt, sym: int) -> np.float32:
    return np.float32(lib().co3o_symbol_value(C.byref(fmt), sym))


# ------------------------------------------------------------------------------------------ convert
def convert(g: np.ndarray, m: np.ndarray, decay: float, fmt: Fmt, want_v: bool = False):
    """One round for one layer.  ``m`` is updated in place.

    Returns dict(sym, ghat, n_saturated, n_nonfinite[, v]).  ``sym`` is uint8 for formats of at
    most 8 bits, uint16 otherwise.
    """
    g = np.ascontiguousarray(g, dtype=np.float32)
    assert m.dtype == np.float32 and m.flags.c_contiguous and m.shape == g.shape
    n = g.size
    wide = 1 + fmt.exp_bits + fmt.mant_bits > 8
    sym = np.empty(n, dtype=np.uint16 if wide else np.uint8)
    ghat = np.empty(n, dtype=np.float32)
    v = np.empty(n, dtype=np.float32) if want_v else None
    nsat, nnf = C.c_uint64(0), C.c_uint64(0)
    st = lib().co3o_convert(_ptr(g), _ptr(m), C.c_float(decay), C.byref(fmt), n,
                            None if wide else _ptr(sym), _ptr(sym) if wide else None, _ptr(ghat), _ptr(v),
                            C.byref(nsat), C.byref(nnf))
    if st != OK:
        raise ValueError("oracle convert: status %d" % st)
    out = dict(sym=sym, ghat=ghat, n_saturated=nsat.value, n_nonfinite=nnf.value)
    if want_v:
        out["v"] = v
    return out


def philox4x32_10(ctr, key) -> np.ndarray:
    """One block of the counter-based generator: four 32-bit words from a 4-word counter and a 2-word key."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    assert c.size == 4 and k.size == 2
    lib().co3o_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def dither_draws(seed: int, client: int, layer: int, first_place: int, n: int) -> np.ndarray:
    """The 24-bit draws of n consecutive elements of one layer of one client, from place first_place on."""
    out = np.empty(n, dtype=np.uint32)
    lib().co3o_dither_draws(seed, client, layer, first_place, n, _ptr(out))
    return out


def convert_dithered(g: np.ndarray, m: np.ndarray, decay: float, fmt: Fmt, draws: np.ndarray):
    """convert() with the dithered rounding rule; draws: one integer in [0, 2^24) per element.  ``m`` is updated."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    d = np.ascontiguousarray(draws, dtype=np.uint32)
    assert m.dtype == np.float32 and m.flags.c_contiguous and m.shape == g.shape and d.shape == g.shape
    n = g.size
    wide = 1 + fmt.exp_bits + fmt.mant_bits > 8
    sym = np.empty(n, dtype=np.uint16 if wide else np.uint8)
    ghat = np.empty(n, dtype=np.float32)
    nsat, nnf = C.c_uint64(0), C.c_uint64(0)
    st = lib().co3o_convert_dithered(_ptr(g), _ptr(m), C.c_float(decay), C.byref(fmt), n, _ptr(d),
                                     None if wide else _ptr(sym), _ptr(sym) if wide else None, _ptr(ghat),
                                     C.byref(nsat), C.byref(nnf))
    if st != OK:
        raise ValueError("oracle convert_dithered: status %d" % st)
    return dict(sym=sym, ghat=ghat, n_saturated=nsat.value, n_nonfinite=nnf.value)


def histogram(sym: np.ndarray) -> np.ndarray:
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    h = np.zeros(256, dtype=np.uint64)
    lib().co3o_histogram(_ptr(sym), sym.size, _ptr(h))
    return h


# ------------------------------------------------------------------------------------------ code
def code_build(weights: np.ndarray, fmt: Fmt) -> Code:
    w = np.ascontiguousarray(weights, dtype=np.uint64)
    assert w.size == 256
    code = Code()
    st = lib().co3o_code_build(_ptr(w), C.byref(fmt), C.byref(code))
    if st != OK:
        raise ValueError("oracle code_build: status %d" % st)
    return code


def code_arrays(code: Code):
    return (np.frombuffer(code.len, dtype=np.uint8).copy(), np.frombuffer(code.bits, dtype=np.uint32).copy())


def make_code(lens, bits) -> Code:
    code = Code()
    for s in range(256):
        code.len[s] = int(lens[s])
        code.bits[s] = int(bits[s])
    return code


# ------------------------------------------------------------------------------------------ streams
def _seg_arr(seg_n_elem):
    return np.ascontiguousarray(seg_n_elem, dtype=np.uint64)


def stream_capacity_bytes(seg_n_elem, chunk_syms: int = 2048, sub_syms: int = 128) -> int:
    seg = _seg_arr(seg_n_elem)
    out = C.c_uint64(0)
    st = lib().co3o_stream_capacity_bytes(_ptr(seg), seg.size, chunk_syms, sub_syms, C.byref(out))
    if st != OK:
        raise ValueError("oracle stream_capacity_bytes: status %d" % st)
    return out.value


def encode(sym: np.ndarray, seg_n_elem, codes, chunk_syms: int = 2048, sub_syms: int = 128,
           capacity: int | None = None):
    """Returns (status, stream bytes as uint8 array trimmed to total_bytes)."""
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    seg = _seg_arr(seg_n_elem)
    assert int(seg.sum()) == sym.size and len(codes) == seg.size
    carr = (Code * max(1, seg.size))(*codes)
    cap = stream_capacity_bytes(seg, chunk_syms, sub_syms) if capacity is None else capacity
    buf = np.full(cap + 64, 0xA5, dtype=np.uint8)  # 64 guard bytes behind the capacity
    used = C.c_uint64(0)
    st = lib().co3o_encode(_ptr(sym), _ptr(seg), carr, seg.size, chunk_syms, sub_syms, _ptr(buf), cap,
                           C.byref(used))
    assert (buf[cap:] == 0xA5).all(), "oracle encoder wrote past the capacity"
    if st != OK:
        return st, None
    return st, buf[:used.value].copy()


def decode(stream: np.ndarray, seg_n_elem, fmts, codes, chunk_syms: int = 2048, sub_syms: int = 128):
    """Returns (status, sym uint8[n], ghat float32[n])."""
    stream = np.ascontiguousarray(stream, dtype=np.uint8)
    seg = _seg_arr(seg_n_elem)
    n = int(seg.sum())
    farr = (Fmt * max(1, seg.size))(*fmts)
    carr = (Code * max(1, seg.size))(*codes)
    sym = np.zeros(n, dtype=np.uint8)
    ghat = np.zeros(n, dtype=np.float32)
    st = lib().co3o_decode(_ptr(stream), stream.size, _ptr(seg), farr, carr, seg.size, chunk_syms, sub_syms,
                           _ptr(sym), _ptr(ghat))
    return st, sym, ghat


def decode_aggregate(streams, seg_n_elem, fmts, codes, chunk_syms: int = 2048, sub_syms: int = 128):
    """Returns (status, avg float32[n])."""
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    seg = _seg_arr(seg_n_elem)
    n = int(seg.sum())
    farr = (Fmt * max(1, seg.size))(*fmts)
    carr = (Code * max(1, seg.size))(*codes)
    ptrs = (C.c_void_p * len(streams))(*[s.ctypes.data for s in streams])
    sizes = np.array([s.size for s in streams], dtype=np.uint64)
    avg = np.zeros(n, dtype=np.float32)
    scratch = np.zeros(max(n, 1), dtype=np.float32)
    st = lib().co3o_decode_aggregate(ptrs, _ptr(sizes), len(streams), _ptr(seg), farr, carr, seg.size,
                                     chunk_syms, sub_syms, _ptr(avg), _ptr(scratch))
    return st, avg


def ps_update(w: np.ndarray, avg: np.ndarray, eta: float) -> None:
    """w <- w - eta * avg in place (float32 arrays of equal size)."""
    assert w.dtype == np.float32 and avg.dtype == np.float32 and w.flags.c_contiguous and avg.flags.c_contiguous
    assert w.size == avg.size
    lib().co3o_ps_update(_ptr(w), _ptr(avg), C.c_float(eta), w.size)


# ------------------------------------------------------------------------------------------ fitting
def gennorm_kurtosis(beta: float) -> float:
    return lib().co3o_gennorm_kurtosis(float(beta))


def gennorm_shape_from_kurtosis(kurt: float, lo: float, hi: float) -> float:
    return lib().co3o_gennorm_shape_from_kurtosis(float(kurt), float(lo), float(hi))


def fit_scale(g: np.ndarray, m, decay: float, log_tab: np.ndarray, beta0: float, dbeta: float):
    """g, m: float32 [n_clients][n] (m may be None).  Returns (status, scale, inv_scale, stats[4])."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    if g.ndim == 1:
        g = g[None, :]
    if m is not None:
        m = np.ascontiguousarray(m, dtype=np.float32).reshape(g.shape)
    tab = np.ascontiguousarray(log_tab, dtype=np.float32)
    sc, inv = C.c_float(0), C.c_float(0)
    stats = np.zeros(4, dtype=np.float64)
    st = lib().co3o_fit_scale(_ptr(g), _ptr(m), C.c_float(decay), g.shape[1], g.shape[0], g.shape[1], _ptr(tab), tab.size,
                              C.c_float(beta0), C.c_float(dbeta), C.byref(sc), C.byref(inv), _ptr(stats))
    return st, sc.value, inv.value, stats


def error_magnitude(g: np.ndarray, m: np.ndarray) -> np.ndarray:
    """[sum |g|, sum |m|] of one layer of one client (float64)."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    m = np.ascontiguousarray(m, dtype=np.float32)
    assert g.shape == m.shape and g.ndim == 1
    out = np.zeros(2, dtype=np.float64)
    lib().co3o_error_magnitude(_ptr(g), _ptr(m), g.size, _ptr(out))
    return out
