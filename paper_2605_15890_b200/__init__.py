"""B200 coded-gradient library: Python binding of the C ABI declared in include/agc.h.

The binding only marshals arguments; every step of the path runs in the CUDA
kernels of libagc.so. There is no CPU fallback: the first use of any entry point
raises ImportError if the shared library has not been built.

The binding is loaded on first attribute access, so that `paper_2605_15890_b200.build`
(which compiles the library) can be imported before the library exists.
"""
import importlib

_BINDING_NAMES = (
    "AGC_CODE_INTERVAL", "AGC_CODE_SUPPORT", "AGC_FLAG_ALLOW_1BIT", "AGC_FLAG_FORCE_DIRECT", "AGC_FLAG_NO_ROW_DECODE",
    "AGC_FLAG_NO_UNBIASED_CHECK", "AGC_STATUS_NONFINITE", "AGC_STATUS_TIMEOUT", "AgcError",
    "AGC_ALLOC_GREEDY", "AGC_ALLOC_RELAXATION", "agc_allocation_upper_bound", "agc_bit_allocate", "agc_bit_allocate_dp", "agc_bit_allocate_heuristic", "agc_code_build", "agc_codes_bytes", "agc_decode",
    "agc_decode_two_track", "agc_decode_update_static", "agc_decode_residuals", "agc_two_track_vector", "AGC_ERR_LIMIT",
    "agc_combine_norm_sums", "agc_encode_norm_sums", "agc_encode_quantize", "agc_encode_quantize_rows", "agc_encode_quantize_with_norms", "agc_eta_balance", "agc_plan_create", "agc_plan_destroy", "agc_plan_encode_layout", "agc_plan_set_first_block", "agc_plan_uses_tma",
    "agc_round_host", "agc_scales_bytes", "agc_selftest_division", "agc_selftest_sqrt", "agc_strerror", "agc_version", "agc_worker_offset",
    "library_path")

__all__ = list(_BINDING_NAMES)


def __getattr__(name):
    if name in _BINDING_NAMES:
        binding = importlib.import_module(".binding", __name__)
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
