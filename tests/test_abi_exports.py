"""The shared library loads without a GPU and exports every function include/co3.h declares; host-only
entry points (status strings, size queries, the Huffman builder) behave as documented."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2204_08211_b200 as co3
from paper_2204_08211_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    return ctypes.CDLL(cuda_build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "co3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(co3_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"co3_encode", "co3_decode_aggregate", "co3_convert", "co3_code_build", "co3_encode_symbols",
            "co3_decode", "co3_workspace_bytes", "co3_stream_capacity_bytes", "co3_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_size_queries():
    assert co3.co3_status_string(co3.OK) == "ok"
    assert len({co3.co3_status_string(i) for i in range(7)}) == 7
    assert "unknown" in co3.co3_status_string(99)
    n, segs = 11_181_642, 62
    cap = co3.co3_stream_capacity_bytes(n, segs)
    assert cap % 16 == 0 and cap >= n * 2                       # 16 bits per element worst case
    # the bound covers the oracle's exact worst case for the same layer layout
    from co3_inputs import RESNET18_LAYER_SIZES
    assert cap >= oracle.stream_capacity_bytes(RESNET18_LAYER_SIZES)
    w0, w10 = co3.co3_workspace_bytes(n, segs, 0), co3.co3_workspace_bytes(n, segs, 10)
    assert w10 > w0 > 0 and w10 - w0 >= 10 * 2 * n
    with pytest.raises(ValueError):
        co3.co3_workspace_bytes(n, segs, 1, chunk_syms=1024)


def test_calls_reject_bad_arguments_without_a_gpu(lib):
    # null pointers and unsupported sizes are refused before any CUDA call is made
    assert lib.co3_encode(None, None, ctypes.c_float(0.9), None, None, None, 1, ctypes.c_uint64(10), 1,
                          ctypes.c_uint64(10), None, ctypes.c_size_t(0), 2048, None, ctypes.c_size_t(0), None,
                          None) == co3.ERR_INVALID_ARG
    assert lib.co3_decode_aggregate(None, ctypes.c_size_t(0), 1, None, None, None, 1, ctypes.c_uint64(10), 2048,
                                    None, None, ctypes.c_size_t(0), None, None) == co3.ERR_INVALID_ARG


@pytest.mark.parametrize("E,M,flush", [(2, 0, 0), (2, 1, 0), (3, 0, 0), (4, 3, 0), (5, 2, 0), (4, 3, 1), (2, 1, 1)])
def test_host_code_builder_equals_oracle(E, M, flush):
    """Two independent constructions (pool of minima vs two queues) must give identical tables."""
    rng = np.random.default_rng(E * 10 + M)
    fmt = co3.make_fmts([(E, M, flush, 1.0, 1.0)])
    ofmt = oracle.make_fmt(E, M, 1.0, bool(flush))
    for t in range(25):
        w = (rng.pareto(0.7, size=256) * rng.choice([1, 10, 1000, 10 ** 6])).astype(np.uint64)
        if t == 0:
            w[:] = 0
        if t == 1:
            w[:] = 5
        if t == 2:                                   # Fibonacci weights: forces the length limit
            a, b = 1, 1
            for i in range(256):
                w[i] = a
                if a + b < 2 ** 54:
                    a, b = b, a + b
        st, code = co3.co3_code_build(w, fmt)
        ln, bits = oracle.code_arrays(oracle.code_build(w, ofmt))
        assert st == co3.OK
        assert np.array_equal(code["len"][0], ln) and np.array_equal(code["bits"][0], bits)
    st, _ = co3.co3_code_build(np.full(256, 2 ** 62, dtype=np.uint64), fmt)
    assert st == co3.ERR_INVALID_ARG
    st, _ = co3.co3_code_build(np.ones(256, dtype=np.uint64), co3.make_fmts([(1, 3, 0, 1.0, 1.0)]))
    assert st == co3.ERR_INVALID_ARG
