"""CO3 uplink pipeline (arXiv 2204.08211) for NVIDIA B200: Python binding of the C-ABI library.

Every function here only marshals arguments for the entry point of the same name in
``include/co3.h``; all computation runs in the CUDA kernels of ``libco3.so``.  There is no CPU
fallback: if the library has not been built, importing a function from it raises.
"""
from .binding import (  # noqa: F401
    CHUNK_SYMS, MAX_CODE_LEN, SUB_SYMS, CODE_DTYPE, FMT_DTYPE, RESULT_DTYPE, SEG_DTYPE,
    ERR_CAPACITY, ERR_CORRUPT, ERR_CUDA, ERR_INVALID_ARG, ERR_NO_CODEWORD, ERR_NONFINITE, OK, FMT_FLUSH_SUBNORMALS,
    co3_code_build, co3_code_build_device, co3_convert, co3_histogram, co3_convert_dither, co3_histogram_dither, co3_encode_dither, co3_convert_static, STATIC_SCRATCH_BYTES, co3_decode, co3_decode_aggregate, co3_decode_aggregate_update, co3_encode, co3_encode_symbols, co3_fit_scale, co3_model_weights, co3_error_magnitude,
    co3_profile_enable, co3_profile_read, co3_status_string, KERNEL_NAMES, co3_stream_capacity_bytes, co3_workspace_bytes,
    library_path, make_fmts, make_segs, to_device, read_results,
)
