"""B200 coded-gradient library: Python binding of the C ABI declared in include/agc.h.

The binding only marshals arguments; every step of the path runs in the CUDA
kernels of libagc.so. There is no CPU fallback: importing `binding` raises if the
shared library has not been built.
"""
from .binding import (  # noqa: F401
    AGC_CODE_INTERVAL, AGC_CODE_SUPPORT, AGC_FLAG_ALLOW_1BIT, AGC_FLAG_FORCE_DIRECT,
    AGC_FLAG_NO_UNBIASED_CHECK, AGC_STATUS_NONFINITE, AGC_STATUS_TIMEOUT, AgcError,
    agc_bit_allocate, agc_bit_allocate_dp, agc_code_build, agc_codes_bytes, agc_decode,
    agc_encode_quantize, agc_plan_create, agc_plan_destroy, agc_plan_uses_tma, agc_round_host,
    agc_scales_bytes, agc_strerror, agc_version, agc_worker_offset, library_path)
