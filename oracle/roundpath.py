"""numpy front end of the C oracle for the per-round path (test infrastructure).

Argument marshalling only; all arithmetic is in agc_oracle.c. Notation follows
the paper's Sec. II with these letters: n workers, k partitions,
d coordinates, bits b_i, bucket size B.
"""
import ctypes as C

import numpy as np

from . import build as _build

BLOCK = 512
STATUS_NONFINITE = 1
STATUS_RANGE = 2

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        u32p, f32p, u8p, i32p = (C.POINTER(C.c_uint32), C.POINTER(C.c_float),
                                 C.POINTER(C.c_uint8), C.POINTER(C.c_int32))
        L.agc_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.agc_oracle_philox4x32_10.restype = None
        L.agc_oracle_uniform15.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64]
        L.agc_oracle_uniform15.restype = C.c_uint32
        L.agc_oracle_quantize_one.argtypes = [C.c_float, C.c_float, C.c_int, C.c_uint32]
        L.agc_oracle_quantize_one.restype = C.c_uint32
        L.agc_oracle_inv_scale.argtypes = [C.c_float, C.c_int]
        L.agc_oracle_inv_scale.restype = C.c_float
        L.agc_oracle_dequantize_one.argtypes = [C.c_uint32, C.c_float, C.c_int]
        L.agc_oracle_dequantize_one.restype = C.c_float
        L.agc_oracle_stream_position.argtypes = [C.c_int64]
        L.agc_oracle_stream_position.restype = C.c_int64
        L.agc_oracle_encode_block.argtypes = [C.c_int, i32p, i32p, f32p, u8p, C.c_int, C.c_uint64,
                                              C.c_uint64, C.c_int64, f32p, u32p, f32p, f32p]
        L.agc_oracle_encode_block.restype = C.c_uint32
        L.agc_oracle_decode_block.argtypes = [C.c_int, u8p, C.c_int, f32p, u8p, u32p, f32p, f32p]
        L.agc_oracle_decode_block.restype = None
        L.agc_oracle_encode_quantize.argtypes = [C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, u8p,
                                                 C.c_int, C.c_uint64, C.c_uint64, f32p, C.c_int64,
                                                 u32p, f32p, f32p]
        L.agc_oracle_encode_quantize.restype = C.c_uint32
        L.agc_oracle_decode.argtypes = [C.c_int, C.c_int64, u8p, C.c_int, f32p, u8p, C.c_int, f32p,
                                        u32p, f32p, f32p, f32p]
        L.agc_oracle_decode.restype = None
        L.agc_oracle_dequantize_worker.argtypes = [C.c_int64, C.c_int, C.c_int, u32p, f32p, f32p]
        L.agc_oracle_dequantize_worker.restype = None
        L.agc_oracle_encode_quantize_global.argtypes = [C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, u8p, C.c_uint64,
                                                        C.c_uint64, f32p, C.c_int64, u32p, f32p, f32p]
        L.agc_oracle_encode_quantize_global.restype = C.c_uint32
        L.agc_oracle_global_sumsq.argtypes = [C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, f32p, C.c_int64, f32p]
        L.agc_oracle_global_sumsq.restype = None
        L.agc_oracle_combine_sumsq.argtypes = [C.c_int, C.c_int, f32p, f32p]
        L.agc_oracle_combine_sumsq.restype = None
        L.agc_oracle_encode_quantize_with_norm.argtypes = [C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, u8p, C.c_uint64,
                                                           C.c_uint64, C.c_int64, f32p, C.c_int64, f32p, u32p, f32p, f32p]
        L.agc_oracle_encode_quantize_with_norm.restype = C.c_uint32
        L.agc_oracle_encode_quantize_grouped.argtypes = [C.c_int, C.c_int, C.c_int64, i32p, i32p, f32p, u8p, C.c_int64,
                                                         C.c_uint64, C.c_uint64, f32p, C.c_int64, u32p, f32p, f32p]
        L.agc_oracle_encode_quantize_grouped.restype = C.c_uint32
        L.agc_oracle_adam_two_track.argtypes = [C.c_int64, f32p, f32p, C.c_float, C.c_float, C.c_float, C.c_float,
                                                C.c_float, C.c_float, C.c_float, C.c_float, f32p, f32p, f32p]
        L.agc_oracle_adam_two_track.restype = None
        _lib = L
    return _lib


def _p(arr, ctype):
    return None if arr is None else arr.ctypes.data_as(C.POINTER(ctype))


def _c(arr, dtype):
    return np.ascontiguousarray(arr, dtype=dtype)


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().agc_oracle_philox4x32_10(_p(ctr, C.c_uint32), _p(key, C.c_uint32), _p(out, C.c_uint32))
    return out


def uniform15(seed, rnd, worker, pos):
    return int(lib().agc_oracle_uniform15(seed, rnd, worker, pos))


def quantize_one(x, inv, b, u):
    """Code of one coordinate for the 15-bit uniform u (before masking to b bits)."""
    return int(lib().agc_oracle_quantize_one(x, inv, b, u))


def inv_scale(S, b):
    return float(lib().agc_oracle_inv_scale(S, b))


def dequantize_one(code, S, b):
    return float(lib().agc_oracle_dequantize_one(code, S, b))


def stream_position(m):
    return int(lib().agc_oracle_stream_position(m))


def num_blocks(d):
    return (d + BLOCK - 1) // BLOCK


def worker_word_offsets(d, bits):
    """Word offset of each worker's message in the concatenation (+ total)."""
    nblk = num_blocks(d)
    off = np.zeros(len(bits) + 1, np.int64)
    off[1:] = np.cumsum(nblk * 16 * np.asarray(bits, np.int64))
    return off


def encode_quantize(row_ptr, col_idx, a, bits, B, seed, rnd, G, d=None, want_x=False):
    """Encode + quantise + pack all workers. G: (k, >=d) float32.
    Returns (codes uint32 [total words], scales float32 [n, nb], status, x or None)."""
    G = np.asarray(G)
    assert G.dtype == np.float32 and G.ndim == 2 and G.strides[1] == 4
    k = G.shape[0]
    d = G.shape[1] if d is None else d
    ld = G.strides[0] // 4
    row_ptr = _c(row_ptr, np.int32)
    col_idx = _c(col_idx, np.int32)
    a = _c(a, np.float32)
    bits = _c(bits, np.uint8)
    n = len(bits)
    off = worker_word_offsets(d, bits)
    nb = (d + B - 1) // B
    codes = np.zeros(int(off[-1]), np.uint32)
    scales = np.zeros((n, nb), np.float32)
    x = np.zeros((n, d), np.float32) if want_x else None
    st = lib().agc_oracle_encode_quantize(n, k, d, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32),
                                          _p(a, C.c_float), _p(bits, C.c_uint8), B, seed, rnd,
                                          _p(G, C.c_float), ld, _p(codes, C.c_uint32),
                                          _p(scales, C.c_float), _p(x, C.c_float))
    return codes, scales, int(st), x


def encode_block(row_ptr, col_idx, a, bits, B, seed, rnd, q, Gblk, want_x=False):
    """One pack block. Gblk: (k, 512) float32, zero beyond d."""
    Gblk = _c(Gblk, np.float32)
    assert Gblk.shape[1] == BLOCK
    row_ptr = _c(row_ptr, np.int32)
    col_idx = _c(col_idx, np.int32)
    a = _c(a, np.float32)
    bits = _c(bits, np.uint8)
    n = len(bits)
    codes = np.zeros(16 * int(bits.astype(np.int64).sum()), np.uint32)
    scales = np.zeros((n, BLOCK // B), np.float32)
    x = np.zeros((n, BLOCK), np.float32) if want_x else None
    st = lib().agc_oracle_encode_block(n, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32),
                                       _p(a, C.c_float), _p(bits, C.c_uint8), B, seed, rnd, q,
                                       _p(Gblk, C.c_float), _p(codes, C.c_uint32),
                                       _p(scales, C.c_float), _p(x, C.c_float))
    return codes, scales, int(st), x


def decode_block(bits, B, w, mask, codes_blk, scales_blk):
    bits = _c(bits, np.uint8)
    w = _c(w, np.float32)
    mask = _c(mask, np.uint8)
    codes_blk = _c(codes_blk, np.uint32)
    scales_blk = _c(scales_blk, np.float32)
    out = np.zeros(BLOCK, np.float32)
    lib().agc_oracle_decode_block(len(bits), _p(bits, C.c_uint8), B, _p(w, C.c_float),
                                  _p(mask, C.c_uint8), _p(codes_blk, C.c_uint32),
                                  _p(scales_blk, C.c_float), _p(out, C.c_float))
    return out


def decode(d, bits, B, w, masks, codes, scales, lr=None, beta=None, want_ghat=True):
    """Masked decode for R realisations. masks: (R, n) uint8. Returns (ghat (R,d) or None,
    beta copy updated or None)."""
    bits = _c(bits, np.uint8)
    w = _c(w, np.float32)
    masks = _c(np.atleast_2d(masks), np.uint8)
    R, n = masks.shape
    assert n == len(bits)
    codes = _c(codes, np.uint32)
    scales = _c(scales, np.float32)
    ghat = np.zeros((R, d), np.float32) if want_ghat else None
    b2 = None
    lr_a = None
    if beta is not None:
        b2 = np.array(beta, dtype=np.float32, copy=True)
        lr_a = _c(lr, np.float32)
        assert lr_a.shape == (R,)
    lib().agc_oracle_decode(n, d, _p(bits, C.c_uint8), B, _p(w, C.c_float), _p(masks, C.c_uint8), R,
                            _p(lr_a, C.c_float), _p(codes, C.c_uint32), _p(scales, C.c_float),
                            _p(ghat, C.c_float), _p(b2, C.c_float))
    return ghat, b2


def dequantize_worker(d, b, B, codes_i, scales_i):
    codes_i = _c(codes_i, np.uint32)
    scales_i = _c(scales_i, np.float32)
    out = np.zeros(d, np.float32)
    lib().agc_oracle_dequantize_worker(d, b, B, _p(codes_i, C.c_uint32), _p(scales_i, C.c_float),
                                       _p(out, C.c_float))
    return out


def adam_constants(b1, b2, step):
    """(1-b1, 1-b2, 1/(1-b1^t), 1/(1-b2^t)) formed in double precision from the fp32 values
    of b1, b2 and rounded to fp32 (t = step >= 1)."""
    b1, b2 = float(np.float32(b1)), float(np.float32(b2))
    return (np.float32(1.0 - b1), np.float32(1.0 - b2), np.float32(1.0 / (1.0 - b1 ** step)),
            np.float32(1.0 / (1.0 - b2 ** step)))


def adam_two_track(gw, gv, lr, b1, b2, eps, step, beta, m, u):
    """One Adam step with first moment from gw and second moment from gv (Sec. V-E).
    Returns updated copies (beta, m, u)."""
    gw, gv = _c(gw, np.float32), _c(gv, np.float32)
    beta, m, u = (np.array(x, dtype=np.float32, copy=True) for x in (beta, m, u))
    c1, c2, ibc1, ibc2 = adam_constants(b1, b2, step)
    lib().agc_oracle_adam_two_track(len(gw), _p(gw, C.c_float), _p(gv, C.c_float), np.float32(lr), np.float32(b1),
                                    np.float32(b2), c1, c2, np.float32(eps), ibc1, ibc2, _p(beta, C.c_float),
                                    _p(m, C.c_float), _p(u, C.c_float))
    return beta, m, u


def encode_quantize_global(row_ptr, col_idx, a, bits, seed, rnd, G, d=None, want_x=False):
    """Encode + quantise + pack with ONE l2 norm per worker (the paper's main formulation).
    Returns (codes uint32, scales float32 [n], status, x or None)."""
    G = np.asarray(G)
    assert G.dtype == np.float32 and G.ndim == 2 and G.strides[1] == 4
    k = G.shape[0]
    d = G.shape[1] if d is None else d
    ld = G.strides[0] // 4
    row_ptr, col_idx = _c(row_ptr, np.int32), _c(col_idx, np.int32)
    a, bits = _c(a, np.float32), _c(bits, np.uint8)
    n = len(bits)
    off = worker_word_offsets(d, bits)
    codes = np.zeros(int(off[-1]), np.uint32)
    scales = np.zeros(n, np.float32)
    x = np.zeros((n, d), np.float32) if want_x else None
    st = lib().agc_oracle_encode_quantize_global(n, k, d, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32),
                                                 _p(a, C.c_float), _p(bits, C.c_uint8), seed, rnd,
                                                 _p(G, C.c_float), ld, _p(codes, C.c_uint32),
                                                 _p(scales, C.c_float), _p(x, C.c_float))
    return codes, scales, int(st), x


def global_sumsq(row_ptr, col_idx, a, G, d=None):
    """Step 1 of the global norm: per-worker sum of squares of the coded vector over the
    coordinates given (a whole vector or a contiguous range of pack blocks). float32 [n]."""
    G = np.asarray(G)
    assert G.dtype == np.float32 and G.ndim == 2 and G.strides[1] == 4
    d = G.shape[1] if d is None else d
    row_ptr, col_idx, a = _c(row_ptr, np.int32), _c(col_idx, np.int32), _c(a, np.float32)
    n = len(row_ptr) - 1
    out = np.zeros(n, np.float32)
    lib().agc_oracle_global_sumsq(n, G.shape[0], d, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32), _p(a, C.c_float),
                                  _p(G, C.c_float), G.strides[0] // 4, _p(out, C.c_float))
    return out


def combine_sumsq(per_range):
    """Sums of squares of consecutive ranges, (ranges, n), combined into the whole vector's."""
    per_range = _c(np.atleast_2d(per_range), np.float32)
    out = np.zeros(per_range.shape[1], np.float32)
    lib().agc_oracle_combine_sumsq(per_range.shape[0], per_range.shape[1], _p(per_range, C.c_float), _p(out, C.c_float))
    return out


def encode_quantize_with_norm(row_ptr, col_idx, a, bits, seed, rnd, G, sumsq, first_block=0, d=None):
    """Step 2 of the global norm on the coordinates given, with the whole vector's sums of
    squares. Returns (codes uint32, scales float32 [n], status)."""
    G = np.asarray(G)
    assert G.dtype == np.float32 and G.ndim == 2 and G.strides[1] == 4
    d = G.shape[1] if d is None else d
    row_ptr, col_idx = _c(row_ptr, np.int32), _c(col_idx, np.int32)
    a, bits, sumsq = _c(a, np.float32), _c(bits, np.uint8), _c(sumsq, np.float32)
    n = len(bits)
    off = worker_word_offsets(d, bits)
    codes = np.zeros(int(off[-1]), np.uint32)
    scales = np.zeros(n, np.float32)
    st = lib().agc_oracle_encode_quantize_with_norm(n, G.shape[0], d, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32),
                                                    _p(a, C.c_float), _p(bits, C.c_uint8), seed, rnd, first_block,
                                                    _p(G, C.c_float), G.strides[0] // 4, _p(sumsq, C.c_float),
                                                    _p(codes, C.c_uint32), _p(scales, C.c_float), None)
    return codes, scales, int(st)


def encode_quantize_grouped(row_ptr, col_idx, a, bits, B, seed, rnd, G, d=None, want_x=False):
    """Encode + quantise + pack with buckets of B = 1024, 2048 or 4096 coordinates (whole groups
    of pack blocks). Returns (codes uint32, scales float32 [n, ceil(d / B)], status, x or None)."""
    assert B % BLOCK == 0 and B >= BLOCK
    G = np.asarray(G)
    assert G.dtype == np.float32 and G.ndim == 2 and G.strides[1] == 4
    k = G.shape[0]
    d = G.shape[1] if d is None else d
    ld = G.strides[0] // 4
    row_ptr, col_idx = _c(row_ptr, np.int32), _c(col_idx, np.int32)
    a, bits = _c(a, np.float32), _c(bits, np.uint8)
    n = len(bits)
    group = B // BLOCK
    nb = (num_blocks(d) + group - 1) // group
    off = worker_word_offsets(d, bits)
    codes = np.zeros(int(off[-1]), np.uint32)
    scales = np.zeros((n, nb), np.float32)
    x = np.zeros((n, d), np.float32) if want_x else None
    st = lib().agc_oracle_encode_quantize_grouped(n, k, d, _p(row_ptr, C.c_int32), _p(col_idx, C.c_int32),
                                                  _p(a, C.c_float), _p(bits, C.c_uint8), group, seed, rnd,
                                                  _p(G, C.c_float), ld, _p(codes, C.c_uint32),
                                                  _p(scales, C.c_float), _p(x, C.c_float))
    return codes, scales, int(st), x


def expand_grouped_scales(scales, d, B):
    """Scales of buckets of B >= 512 coordinates as an (n, nblk) array for decode() with B = 512."""
    group = B // BLOCK
    return np.ascontiguousarray(np.repeat(np.asarray(scales, np.float32), group, axis=1)[:, :num_blocks(d)])


def expand_global_scales(scales, d):
    """The per-worker global scales as an (n, nblk) array for decode() with B = 512."""
    return np.repeat(np.asarray(scales, np.float32)[:, None], num_blocks(d), axis=1)
