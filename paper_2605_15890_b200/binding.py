"""ctypes binding of libagc.so, one Python function per C entry point, same names.

Host arrays are numpy arrays; device buffers are passed as torch CUDA tensors (or
raw integer addresses); streams as torch.cuda.Stream, an integer handle or None
(the current torch stream).
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libagc.so")

AGC_FLAG_ALLOW_1BIT = 1
AGC_FLAG_NO_UNBIASED_CHECK = 2
AGC_FLAG_FORCE_DIRECT = 4
AGC_FLAG_NO_ROW_DECODE = 8
AGC_STATUS_NONFINITE = 1
AGC_STATUS_TIMEOUT = 4
AGC_CODE_INTERVAL = 0
AGC_CODE_SUPPORT = 1
AGC_ALLOC_GREEDY = 0
AGC_ALLOC_RELAXATION = 1
AGC_ERR_LIMIT = -10


class AgcAdam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("step", C.c_int64)]


class AgcError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"agc error {code}: {text}")
        self.code = code


def library_path():
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2605_15890_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, i32p, f32p, f64p, u8p, u32p = (C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float),
                                       C.POINTER(C.c_double), C.POINTER(C.c_uint8),
                                       C.POINTER(C.c_uint32))
    L.agc_plan_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, f32p,
                                  f32p, u8p, C.c_uint32, C.c_uint64, C.c_uint32]
    L.agc_plan_create.restype = C.c_int
    L.agc_plan_destroy.argtypes = [vp]
    L.agc_plan_destroy.restype = None
    for name in ("agc_codes_bytes", "agc_scales_bytes"):
        getattr(L, name).argtypes = [vp]
        getattr(L, name).restype = C.c_size_t
    L.agc_worker_offset.argtypes = [vp, C.c_int]
    L.agc_worker_offset.restype = C.c_size_t
    L.agc_plan_set_first_block.argtypes = [vp, C.c_int64]
    L.agc_plan_set_first_block.restype = C.c_int
    L.agc_plan_uses_tma.argtypes = [vp]
    L.agc_plan_uses_tma.restype = C.c_int
    L.agc_encode_quantize.argtypes = [vp, vp, C.c_int64, C.c_uint64, vp, vp, vp, vp]
    L.agc_encode_quantize.restype = C.c_int
    L.agc_encode_quantize_rows.argtypes = [vp, vp, C.c_uint64, vp, vp, vp, vp]
    L.agc_encode_quantize_rows.restype = C.c_int
    L.agc_plan_encode_layout.argtypes = [vp, i32p]
    L.agc_plan_encode_layout.restype = C.c_int
    L.agc_encode_norm_sums.argtypes = [vp, vp, C.c_int64, vp, vp]
    L.agc_encode_norm_sums.restype = C.c_int
    L.agc_combine_norm_sums.argtypes = [C.c_int, C.c_int, f32p, f32p]
    L.agc_combine_norm_sums.restype = C.c_int
    L.agc_encode_quantize_with_norms.argtypes = [vp, vp, C.c_int64, C.c_uint64, vp, vp, vp, vp, vp]
    L.agc_encode_quantize_with_norms.restype = C.c_int
    L.agc_decode.argtypes = [vp, vp, vp, vp, C.c_int, f32p, vp, vp, vp, vp]
    L.agc_decode.restype = C.c_int
    L.agc_decode_update_static.argtypes = [C.c_int, C.c_int64, C.c_uint32, u8p, f32p, vp, vp, vp, C.c_int, f32p,
                                           vp, vp]
    L.agc_decode_update_static.restype = C.c_int
    L.agc_decode_residuals.argtypes = [vp, vp, vp, vp, C.c_int, vp, vp, vp]
    L.agc_decode_residuals.restype = C.c_int
    L.agc_decode_two_track.argtypes = [vp, vp, vp, vp, f32p, vp, vp, vp, vp, vp, C.POINTER(AgcAdam), vp, vp]
    L.agc_decode_two_track.restype = C.c_int
    L.agc_two_track_vector.argtypes = [C.c_int, C.c_int, f64p, u8p, C.c_double, C.c_double, C.c_double, i32p, f32p,
                                       f32p]
    L.agc_two_track_vector.restype = C.c_int
    L.agc_round_host.argtypes = [vp, vp, C.c_int64, C.c_uint64, vp, vp, u32p, vp]
    L.agc_round_host.restype = C.c_int
    for name in ("agc_bit_allocate", "agc_bit_allocate_dp"):
        getattr(L, name).argtypes = [C.c_int, f64p, C.c_int, C.c_int, C.c_int, C.c_double, C.c_double,
                                     u8p, f64p]
        getattr(L, name).restype = C.c_int
    L.agc_code_build.argtypes = [C.c_int, C.c_int, f64p, u8p, C.c_double, C.c_double, C.c_int, i32p,
                                 i32p, C.c_int32, i32p, i32p, f32p, f32p, f64p]
    L.agc_code_build.restype = C.c_int
    L.agc_selftest_division.argtypes = [C.POINTER(C.c_ulonglong)]
    L.agc_selftest_division.restype = C.c_int
    L.agc_selftest_sqrt.argtypes = [C.POINTER(C.c_ulonglong)]
    L.agc_selftest_sqrt.restype = C.c_int
    L.agc_bit_allocate_heuristic.argtypes = [C.c_int, C.c_int, f64p, C.c_int, C.c_int, C.c_int, C.c_double, C.c_double,
                                             u8p, f64p]
    L.agc_bit_allocate_heuristic.restype = C.c_int
    L.agc_allocation_upper_bound.argtypes = [C.c_int, f64p, C.c_int, C.c_int, C.c_int, C.c_double, C.c_double, f64p]
    L.agc_allocation_upper_bound.restype = C.c_int
    L.agc_eta_balance.argtypes = [C.c_int, f64p, C.c_int, C.c_double, f64p]
    L.agc_eta_balance.restype = C.c_int
    L.agc_strerror.argtypes = [C.c_int]
    L.agc_strerror.restype = C.c_char_p
    L.agc_version.argtypes = []
    L.agc_version.restype = C.c_int
    return L


_lib = _load()


def _check(rc):
    if rc != 0:
        raise AgcError(rc, _lib.agc_strerror(rc).decode())


def _np(arr, dtype):
    return np.ascontiguousarray(arr, dtype=dtype)


def _hp(arr, ctype):
    return None if arr is None else arr.ctypes.data_as(C.POINTER(ctype))


def _dev(x):
    """Device (or pinned host) address of a torch tensor / integer / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return C.c_void_p(x)
    return C.c_void_p(x.data_ptr())


def _stream(s):
    if s is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(s, int):
        return C.c_void_p(s)
    return C.c_void_p(s.cuda_stream)


def agc_strerror(code):
    return _lib.agc_strerror(code).decode()


def agc_version():
    return _lib.agc_version()


def agc_plan_create(n_workers, k_parts, d, row_ptr, col_idx, a, w, p, bits, bucket, seed, flags=0):
    """Returns an opaque plan handle (free it with agc_plan_destroy)."""
    row_ptr, col_idx = _np(row_ptr, np.int32), _np(col_idx, np.int32)
    a, w, p, bits = _np(a, np.float32), _np(w, np.float32), _np(p, np.float32), _np(bits, np.uint8)
    if len(row_ptr) != n_workers + 1 or len(w) != n_workers or len(p) != n_workers or \
            len(bits) != n_workers or len(col_idx) != len(a) or len(a) < int(row_ptr[-1]):
        raise AgcError(-1, "array lengths do not match n_workers / nnz")
    h = C.c_void_p()
    _check(_lib.agc_plan_create(C.byref(h), n_workers, k_parts, d, _hp(row_ptr, C.c_int32),
                                _hp(col_idx, C.c_int32), _hp(a, C.c_float), _hp(w, C.c_float),
                                _hp(p, C.c_float), _hp(bits, C.c_uint8), bucket, seed, flags))
    return h


def agc_plan_destroy(plan):
    _lib.agc_plan_destroy(plan)


def agc_codes_bytes(plan):
    return _lib.agc_codes_bytes(plan)


def agc_scales_bytes(plan):
    return _lib.agc_scales_bytes(plan)


def agc_worker_offset(plan, i):
    return _lib.agc_worker_offset(plan, i)


def agc_plan_set_first_block(plan, first_block):
    _check(_lib.agc_plan_set_first_block(plan, first_block))


def agc_plan_uses_tma(plan):
    return bool(_lib.agc_plan_uses_tma(plan))


def agc_encode_quantize(plan, G_dev, ld, rnd, codes_dev, scales_dev, status_dev=None, stream=None):
    _check(_lib.agc_encode_quantize(plan, _dev(G_dev), ld, rnd, _dev(codes_dev), _dev(scales_dev),
                                    _dev(status_dev), _stream(stream)))


def agc_encode_quantize_rows(plan, G_rows_dev, rnd, codes_dev, scales_dev, status_dev=None, stream=None):
    """G_rows_dev: device array of k row addresses (a torch int64 CUDA tensor)."""
    _check(_lib.agc_encode_quantize_rows(plan, _dev(G_rows_dev), rnd, _dev(codes_dev), _dev(scales_dev),
                                         _dev(status_dev), _stream(stream)))


def agc_plan_encode_layout(plan):
    """dict(staged, groups, rows_staged, stages) of the plan's encoder tiling."""
    out = np.zeros(4, np.int32)
    _check(_lib.agc_plan_encode_layout(plan, _hp(out, C.c_int32)))
    return {"staged": bool(out[0]), "groups": int(out[1]), "rows_staged": int(out[2]), "stages": int(out[3])}


def agc_encode_norm_sums(plan, G_dev, ld, sumsq_dev, stream=None):
    """First pass of the global-norm encoder over the plan's coordinates: n sums of squares."""
    _check(_lib.agc_encode_norm_sums(plan, _dev(G_dev), ld, _dev(sumsq_dev), _stream(stream)))


def agc_combine_norm_sums(per_range):
    """per_range: (ranges, n) float32 host array in range order; returns the combined sums [n]."""
    per_range = np.ascontiguousarray(np.atleast_2d(per_range), np.float32)
    out = np.zeros(per_range.shape[1], np.float32)
    _check(_lib.agc_combine_norm_sums(per_range.shape[0], per_range.shape[1], _hp(per_range, C.c_float),
                                      _hp(out, C.c_float)))
    return out


def agc_encode_quantize_with_norms(plan, G_dev, ld, rnd, sumsq_dev, codes_dev, scales_dev, status_dev=None,
                                   stream=None):
    """Second pass of the global-norm encoder with the whole vector's sums of squares."""
    _check(_lib.agc_encode_quantize_with_norms(plan, _dev(G_dev), ld, rnd, _dev(sumsq_dev), _dev(codes_dev),
                                               _dev(scales_dev), _dev(status_dev), _stream(stream)))


def agc_decode(plan, codes_dev, scales_dev, masks_dev, R, lr_host=None, ghat_dev=None, beta_dev=None,
               status_dev=None, stream=None):
    lr = None if lr_host is None else _np(lr_host, np.float32)
    if lr is not None and lr.size < R:
        raise AgcError(-1, "lr_host shorter than R")
    _check(_lib.agc_decode(plan, _dev(codes_dev), _dev(scales_dev), _dev(masks_dev), R,
                           _hp(lr, C.c_float), _dev(ghat_dev), _dev(beta_dev), _dev(status_dev),
                           _stream(stream)))


def agc_decode_residuals(plan, codes_dev, scales_dev, masks_dev, R, g_ref_dev, sqerr_dev, stream=None):
    """sqerr_dev: device float64 [R], overwritten with ||g_hat^(r) - g_ref||^2."""
    _check(_lib.agc_decode_residuals(plan, _dev(codes_dev), _dev(scales_dev), _dev(masks_dev), R,
                                     _dev(g_ref_dev), _dev(sqerr_dev), _stream(stream)))


def agc_decode_update_static(n_workers, d, bucket, bits, w, codes_dev, scales_dev, masks_dev, R, lr_host,
                             beta_dev, stream=None):
    """Multi-realisation fused update that allocates nothing (its scratch is a fixed array
    inside the library). bits / w / lr_host are host arrays; the rest are device buffers."""
    bits, w, lr = _np(bits, np.uint8), _np(w, np.float32), _np(lr_host, np.float32)
    if len(bits) != n_workers or len(w) != n_workers or lr.size < R:
        raise AgcError(-1, "array lengths do not match n_workers / R")
    _check(_lib.agc_decode_update_static(n_workers, d, bucket, _hp(bits, C.c_uint8), _hp(w, C.c_float),
                                         _dev(codes_dev), _dev(scales_dev), _dev(masks_dev), R,
                                         _hp(lr, C.c_float), _dev(beta_dev), _stream(stream)))


def agc_decode_two_track(plan, codes_dev, scales_dev, mask_dev, v_host, ghat_w_dev=None, ghat_v_dev=None,
                         beta_dev=None, m_dev=None, u_dev=None, adam=None, status_dev=None, stream=None):
    """adam: (lr, beta1, beta2, eps, step) or None."""
    v = _np(v_host, np.float32)
    ad = None if adam is None else AgcAdam(float(adam[0]), float(adam[1]), float(adam[2]), float(adam[3]), int(adam[4]))
    _check(_lib.agc_decode_two_track(plan, _dev(codes_dev), _dev(scales_dev), _dev(mask_dev), _hp(v, C.c_float),
                                     _dev(ghat_w_dev), _dev(ghat_v_dev), _dev(beta_dev), _dev(m_dev), _dev(u_dev),
                                     None if ad is None else C.byref(ad), _dev(status_dev), _stream(stream)))


def agc_two_track_vector(n, k, p, bits, phi_dim, row_ptr, a, eta=1.0, lam=1.0):
    """Returns v* float32 [n] (Sec. V-E)."""
    p, bits = _np(p, np.float64), _np(bits, np.uint8)
    row_ptr, a = _np(row_ptr, np.int32), _np(a, np.float32)
    v = np.zeros(n, np.float32)
    _check(_lib.agc_two_track_vector(n, k, _hp(p, C.c_double), _hp(bits, C.c_uint8), phi_dim, eta, lam,
                                     _hp(row_ptr, C.c_int32), _hp(a, C.c_float), _hp(v, C.c_float)))
    return v


def agc_round_host(plan, G_host, ld_host, rnd, mask_host, ghat_host, stream=None):
    """G_host / mask_host / ghat_host: torch CPU tensors (pinned recommended) or numpy
    arrays. Returns the status bits of the round."""
    def addr(x):
        if isinstance(x, np.ndarray):
            return C.c_void_p(x.ctypes.data)
        return C.c_void_p(x.data_ptr())
    st = C.c_uint32(0)
    _check(_lib.agc_round_host(plan, addr(G_host), ld_host, rnd, addr(mask_host), addr(ghat_host),
                               C.byref(st), _stream(stream)))
    return st.value


def agc_eta_balance(p, z_tot, phi_dim):
    p = _np(p, np.float64)
    eta = C.c_double(0.0)
    _check(_lib.agc_eta_balance(len(p), _hp(p, C.c_double), z_tot, phi_dim, C.byref(eta)))
    return eta.value


def agc_selftest_division():
    """Number of (numerator, scale) pairs for which the encoder's division differs from the
    correctly rounded quotient (expected 0)."""
    bad = C.c_ulonglong(0)
    _check(_lib.agc_selftest_division(C.byref(bad)))
    return bad.value


def agc_selftest_sqrt():
    """Number of normal floats whose square root in the encoder differs from the correctly
    rounded one (expected 0)."""
    bad = C.c_ulonglong(0)
    _check(_lib.agc_selftest_sqrt(C.byref(bad)))
    return bad.value


def _alloc(fn, p, z_tot, b_min, b_max, phi_dim, eta):
    p = _np(p, np.float64)
    bits = np.zeros(len(p), np.uint8)
    F = C.c_double(0.0)
    _check(fn(len(p), _hp(p, C.c_double), z_tot, b_min, b_max, phi_dim, eta, _hp(bits, C.c_uint8),
              C.byref(F)))
    return bits, F.value


def agc_bit_allocate(p, z_tot, b_min=2, b_max=8, phi_dim=512.0, eta=1.0):
    """Returns (bits uint8 [n], F)."""
    return _alloc(_lib.agc_bit_allocate, p, z_tot, b_min, b_max, phi_dim, eta)


def agc_bit_allocate_dp(p, z_tot, b_min=2, b_max=8, phi_dim=512.0, eta=1.0):
    return _alloc(_lib.agc_bit_allocate_dp, p, z_tot, b_min, b_max, phi_dim, eta)


def agc_bit_allocate_heuristic(method, p, z_tot, b_min=2, b_max=8, phi_dim=512.0, eta=1.0):
    """The greedy (AGC_ALLOC_GREEDY) or continuous-relaxation (AGC_ALLOC_RELAXATION) heuristic of
    the allocator comparison. Returns (bits uint8 [n], F)."""
    p = _np(p, np.float64)
    bits = np.zeros(len(p), np.uint8)
    F = C.c_double(0.0)
    _check(_lib.agc_bit_allocate_heuristic(method, len(p), _hp(p, C.c_double), z_tot, b_min, b_max, phi_dim, eta,
                                           _hp(bits, C.c_uint8), C.byref(F)))
    return bits, F.value


def agc_allocation_upper_bound(p, z_tot, b_min=2, b_max=8, phi_dim=512.0, eta=1.0):
    p = _np(p, np.float64)
    bound = C.c_double(0.0)
    _check(_lib.agc_allocation_upper_bound(len(p), _hp(p, C.c_double), z_tot, b_min, b_max, phi_dim, eta, C.byref(bound)))
    return bound.value


def agc_code_build(n, k, p, bits, phi_dim, eta=1.0, mode=AGC_CODE_INTERVAL, sup_row_ptr=None,
                   sup_col_idx=None):
    """Returns (row_ptr int32 [n+1], col_idx int32 [nnz], a float32 [nnz], w float32 [n], Y float64 [n])."""
    p, bits = _np(p, np.float64), _np(bits, np.uint8)
    if mode == AGC_CODE_SUPPORT:
        sup_row_ptr, sup_col_idx = _np(sup_row_ptr, np.int32), _np(sup_col_idx, np.int32)
        cap = int(sup_row_ptr[-1])
    else:
        cap = n + k
    row_ptr = np.zeros(n + 1, np.int32)
    col = np.zeros(cap, np.int32)
    a = np.zeros(cap, np.float32)
    w = np.zeros(n, np.float32)
    Y = np.zeros(n, np.float64)
    _check(_lib.agc_code_build(n, k, _hp(p, C.c_double), _hp(bits, C.c_uint8), phi_dim, eta, mode,
                               _hp(sup_row_ptr, C.c_int32), _hp(sup_col_idx, C.c_int32), cap,
                               _hp(row_ptr, C.c_int32), _hp(col, C.c_int32), _hp(a, C.c_float),
                               _hp(w, C.c_float), _hp(Y, C.c_double)))
    nnz = int(row_ptr[-1])
    return row_ptr, col[:nnz].copy(), a[:nnz].copy(), w, Y
