"""numpy-facing wrapper of the scalar C oracle (oracle/mqg_oracle.c).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU-baseline
leg import this module; the product package never does.  Each function forwards to
the C function of the same name and only marshals arguments; the arithmetic and the
citations live in the C file.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u64, _u32, _int = C.c_uint64, C.c_uint32, C.c_int
_vp = C.c_void_p


def _ptr(a):
    return a.ctypes.data_as(_vp)


def _decl(name, restype, *argtypes):
    f = getattr(_lib, name)
    f.restype = restype
    f.argtypes = list(argtypes)
    return f


_philox = _decl("mqo_philox4x32_10", None, _vp, _vp, _vp)
_draw_h = _decl("mqo_draw_h", None, _u64, _u32, _u32, _u64, _u64, _vp)
_widen = _decl("mqo_widen_bf16", None, _vp, _u64, _vp)
_scales = _decl("mqo_bucket_scales", None, _vp, _u64, _u64, _vp)
_encode = _decl("mqo_encode", None, _vp, _u64, _int, _u64, _vp, _vp, _vp)
_pack = _decl("mqo_pack", None, _vp, _u64, _int, _vp)
_unpack = _decl("mqo_unpack", None, _vp, _u64, _int, _vp)
_dequant = _decl("mqo_dequantize", None, _vp, _u64, _int, _u64, _vp, _vp)
_apply = _decl("mqo_apply", None, _vp, _vp, C.c_float, _u64)
_quantize = _decl("mqo_quantize", _int, _vp, _u64, _int, _u64, _u64, _vp, _vp, _int, _u32,
                  _u32, _u64)
_deq_acc = _decl("mqo_dequant_accumulate", _int, _vp, _vp, _int, _int, _u64, _vp, _u64, _int)
_server = _decl("mqo_server_step", _int, _vp, _vp, _int, _int, _u64, _u64, _vp, C.c_float, _vp)
_requant = _decl("mqo_server_requantize", _int, _vp, _vp, _int, _int, _u64, _u64, C.c_float, _u64, _vp, _vp,
                _u32, _u32)
_qseg = _decl("mqo_quantize_segments", _int, _vp, _int, _vp, _vp, _int, _u64, _vp, _vp, _int,
              _u32, _u32, _u64)
_sseg = _decl("mqo_server_step_segments", _int, _vp, _vp, _int, _int, _int, _vp, _vp, _vp,
              C.c_float, _vp)


def code_words(n, bits):
    return (int(n) * int(bits) + 31) // 32


def num_buckets(n, bucket):
    return (int(n) + int(bucket) - 1) // int(bucket)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    _philox(_ptr(ctr), _ptr(key), _ptr(out))
    return out


def draw_h(seed, worker, step, elem_offset, n):
    h = np.empty(n, np.uint16)
    _draw_h(seed, worker, step, elem_offset, n, _ptr(h))
    return h


def widen_bf16(x_u16):
    x_u16 = _c(x_u16, np.uint16)
    out = np.empty(x_u16.size, np.float32)
    _widen(_ptr(x_u16), x_u16.size, _ptr(out))
    return out


def bucket_scales(x, bucket):
    x = _c(x, np.float32)
    s = np.empty(num_buckets(x.size, bucket), np.float32)
    _scales(_ptr(x), x.size, bucket, _ptr(s))
    return s


def encode(x, bits, bucket, scales, h):
    x = _c(x, np.float32)
    scales = _c(scales, np.float32)
    h = _c(h, np.uint16)
    assert h.size == x.size and scales.size == num_buckets(x.size, bucket)
    q = np.empty(x.size, np.uint8)
    _encode(_ptr(x), x.size, bits, bucket, _ptr(scales), _ptr(h), _ptr(q))
    return q


def pack(q, bits):
    q = _c(q, np.uint8)
    words = np.empty(code_words(q.size, bits), np.uint32)
    _pack(_ptr(q), q.size, bits, _ptr(words))
    return words


def unpack(words, n, bits):
    words = _c(words, np.uint32)
    assert words.size >= code_words(n, bits)
    q = np.empty(n, np.uint8)
    _unpack(_ptr(words), n, bits, _ptr(q))
    return q


def dequantize(q, bits, bucket, scales):
    q = _c(q, np.uint8)
    scales = _c(scales, np.float32)
    xhat = np.empty(q.size, np.float32)
    _dequant(_ptr(q), q.size, bits, bucket, _ptr(scales), _ptr(xhat))
    return xhat


def apply(params, acc, lr):
    """In place on `params` (float32, contiguous)."""
    assert params.dtype == np.float32 and params.flags.c_contiguous
    acc = _c(acc, np.float32)
    _apply(_ptr(params), _ptr(acc), lr, params.size)
    return params


def quantize(grad, bits, bucket, seed, worker=0, step=0, elem_offset=0, dtype="f32"):
    """grad: float32 array, or uint16 array of bf16 bit patterns when dtype == 'bf16'."""
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    n = grad.size
    codes = np.zeros(code_words(n, bits), np.uint32)
    scales = np.zeros(num_buckets(n, bucket) if n else 0, np.float32)
    rc = _quantize(_ptr(grad), n, bits, bucket, seed, _ptr(codes), _ptr(scales),
                   1 if dtype == "bf16" else 0, worker, step, elem_offset)
    if rc:
        raise ValueError("mqo_quantize failed: %d" % rc)
    return codes, scales


def _ptr_array(arrs, dtype):
    arrs = [_c(a, dtype) for a in arrs]
    tab = (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    return arrs, tab


def dequant_accumulate(codes, scales, bits, n, bucket, acc=None):
    """Returns acc; when `acc` is given the sum is added into a copy of it."""
    W = len(codes)
    codes, ctab = _ptr_array(codes, np.uint32)
    scales, stab = _ptr_array(scales, np.float32)
    add = acc is not None
    out = np.array(acc, np.float32, copy=True) if add else np.empty(n, np.float32)
    rc = _deq_acc(ctab, stab, W, bits, n, _ptr(out), bucket, 1 if add else 0)
    if rc:
        raise ValueError("mqo_dequant_accumulate failed: %d" % rc)
    return out


def server_step(codes, scales, bits, n, bucket, params, lr, want_acc=False):
    """In place on `params`; returns (params, acc or None)."""
    assert params.dtype == np.float32 and params.flags.c_contiguous and params.size == n
    W = len(codes)
    codes, ctab = _ptr_array(codes, np.uint32)
    scales, stab = _ptr_array(scales, np.float32)
    acc = np.empty(n, np.float32) if want_acc else None
    rc = _server(ctab, stab, W, bits, n, bucket, _ptr(params), lr,
                 _ptr(acc) if want_acc else None)
    if rc:
        raise ValueError("mqo_server_step failed: %d" % rc)
    return params, acc


def server_requantize(codes, scales, bits, n, bucket, mean_scale, seed, worker=0, step=0):
    W = len(codes)
    codes, ctab = _ptr_array(codes, np.uint32)
    scales, stab = _ptr_array(scales, np.float32)
    out_c = np.zeros(code_words(n, bits), np.uint32)
    out_s = np.zeros(num_buckets(n, bucket) if n else 0, np.float32)
    rc = _requant(ctab, stab, W, bits, n, bucket, mean_scale, seed, _ptr(out_c), _ptr(out_s), worker, step)
    if rc:
        raise ValueError("mqo_server_requantize failed: %d" % rc)
    return out_c, out_s


def quantize_segments(grad, seg_off, code_off, bits, seed, worker=0, step=0, elem_offset=0,
                      dtype="f32"):
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    seg_off = _c(seg_off, np.uint64)
    code_off = _c(code_off, np.uint64)
    nseg = seg_off.size - 1
    codes = np.zeros(int(code_off[-1]), np.uint32)
    scales = np.zeros(nseg, np.float32)
    rc = _qseg(_ptr(grad), nseg, _ptr(seg_off), _ptr(code_off), bits, seed, _ptr(codes),
               _ptr(scales), 1 if dtype == "bf16" else 0, worker, step, elem_offset)
    if rc:
        raise ValueError("mqo_quantize_segments failed: %d" % rc)
    return codes, scales


def server_step_segments(codes, scales, bits, seg_off, code_off, params, lr, want_acc=False):
    assert params.dtype == np.float32 and params.flags.c_contiguous
    W = len(codes)
    seg_off = _c(seg_off, np.uint64)
    code_off = _c(code_off, np.uint64)
    codes, ctab = _ptr_array(codes, np.uint32)
    scales, stab = _ptr_array(scales, np.float32)
    acc = np.zeros(params.size, np.float32) if want_acc else None
    rc = _sseg(ctab, stab, W, bits, seg_off.size - 1, _ptr(seg_off), _ptr(code_off),
               _ptr(params), lr, _ptr(acc) if want_acc else None)
    if rc:
        raise ValueError("mqo_server_step_segments failed: %d" % rc)
    return params, acc


# ---- codec variant: (min, max) range with nearest rounding ---------------------------------
_ranges = _decl("mqo_bucket_ranges", None, _vp, _u64, _u64, _vp)
_encode_mm = _decl("mqo_encode_minmax", None, _vp, _u64, _int, _u64, _vp, _vp)
_dequant_mm = _decl("mqo_dequantize_minmax", None, _vp, _u64, _int, _u64, _vp, _vp)
_quantize_mm = _decl("mqo_quantize_minmax", _int, _vp, _u64, _int, _u64, _vp, _vp, _int)
_deq_acc_mm = _decl("mqo_dequant_accumulate_minmax", _int, _vp, _vp, _int, _int, _u64, _vp, _u64, _int)
_server_mm = _decl("mqo_server_step_minmax", _int, _vp, _vp, _int, _int, _u64, _u64, _vp, C.c_float, _vp)


def bucket_ranges(x, bucket):
    """(lo, hi) per bucket, interleaved: ranges[2k] = lo, ranges[2k + 1] = hi."""
    x = _c(x, np.float32)
    r = np.empty(2 * num_buckets(x.size, bucket), np.float32)
    _ranges(_ptr(x), x.size, bucket, _ptr(r))
    return r


def encode_minmax(x, bits, bucket, ranges):
    x = _c(x, np.float32)
    ranges = _c(ranges, np.float32)
    assert ranges.size == 2 * num_buckets(x.size, bucket)
    q = np.empty(x.size, np.uint8)
    _encode_mm(_ptr(x), x.size, bits, bucket, _ptr(ranges), _ptr(q))
    return q


def dequantize_minmax(q, bits, bucket, ranges):
    q = _c(q, np.uint8)
    ranges = _c(ranges, np.float32)
    xhat = np.empty(q.size, np.float32)
    _dequant_mm(_ptr(q), q.size, bits, bucket, _ptr(ranges), _ptr(xhat))
    return xhat


def quantize_minmax(grad, bits, bucket, dtype="f32"):
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    n = grad.size
    codes = np.zeros(code_words(n, bits), np.uint32)
    ranges = np.zeros(2 * num_buckets(n, bucket) if n else 0, np.float32)
    rc = _quantize_mm(_ptr(grad), n, bits, bucket, _ptr(codes), _ptr(ranges), 1 if dtype == "bf16" else 0)
    if rc:
        raise ValueError("mqo_quantize_minmax failed: %d" % rc)
    return codes, ranges


def dequant_accumulate_minmax(codes, ranges, bits, n, bucket, acc=None):
    W = len(codes)
    codes, ctab = _ptr_array(codes, np.uint32)
    ranges, rtab = _ptr_array(ranges, np.float32)
    add = acc is not None
    out = np.array(acc, np.float32, copy=True) if add else np.empty(n, np.float32)
    rc = _deq_acc_mm(ctab, rtab, W, bits, n, _ptr(out), bucket, 1 if add else 0)
    if rc:
        raise ValueError("mqo_dequant_accumulate_minmax failed: %d" % rc)
    return out


def server_step_minmax(codes, ranges, bits, n, bucket, params, lr, want_acc=False):
    assert params.dtype == np.float32 and params.flags.c_contiguous and params.size == n
    W = len(codes)
    codes, ctab = _ptr_array(codes, np.uint32)
    ranges, rtab = _ptr_array(ranges, np.float32)
    acc = np.empty(n, np.float32) if want_acc else None
    rc = _server_mm(ctab, rtab, W, bits, n, bucket, _ptr(params), lr, _ptr(acc) if want_acc else None)
    if rc:
        raise ValueError("mqo_server_step_minmax failed: %d" % rc)
    return params, acc


# ---- codec variant: L2-norm scale -----------------------------------------------------------
_sumsq = _decl("mqo_sumsq_tree", C.c_float, _vp, _u64)
_norms = _decl("mqo_bucket_norms", None, _vp, _u64, _u64, _vp)
_quantize_l2 = _decl("mqo_quantize_l2", _int, _vp, _u64, _int, _u64, _u64, _vp, _vp, _int, _u32,
                     _u32, _u64)
_qseg_l2 = _decl("mqo_quantize_segments_l2", _int, _vp, _int, _vp, _vp, _int, _u64, _vp, _vp, _int,
                 _u32, _u32, _u64)


def sumsq_tree(x):
    """The fixed-order fp32 sum of squares of one bucket (as a numpy float32)."""
    x = _c(x, np.float32)
    return np.float32(_sumsq(_ptr(x), x.size))


def bucket_norms(x, bucket):
    x = _c(x, np.float32)
    s = np.empty(num_buckets(x.size, bucket), np.float32)
    _norms(_ptr(x), x.size, bucket, _ptr(s))
    return s


def quantize_l2(grad, bits, bucket, seed, worker=0, step=0, elem_offset=0, dtype="f32"):
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    n = grad.size
    codes = np.zeros(code_words(n, bits), np.uint32)
    scales = np.zeros(num_buckets(n, bucket) if n else 0, np.float32)
    rc = _quantize_l2(_ptr(grad), n, bits, bucket, seed, _ptr(codes), _ptr(scales),
                      1 if dtype == "bf16" else 0, worker, step, elem_offset)
    if rc:
        raise ValueError("mqo_quantize_l2 failed: %d" % rc)
    return codes, scales


def quantize_segments_l2(grad, seg_off, code_off, bits, seed, worker=0, step=0, elem_offset=0,
                         dtype="f32"):
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    seg_off = _c(seg_off, np.uint64)
    code_off = _c(code_off, np.uint64)
    nseg = seg_off.size - 1
    codes = np.zeros(int(code_off[-1]), np.uint32)
    scales = np.zeros(nseg, np.float32)
    rc = _qseg_l2(_ptr(grad), nseg, _ptr(seg_off), _ptr(code_off), bits, seed, _ptr(codes),
                  _ptr(scales), 1 if dtype == "bf16" else 0, worker, step, elem_offset)
    if rc:
        raise ValueError("mqo_quantize_segments_l2 failed: %d" % rc)
    return codes, scales


# ---- codec variant: one bit per element with error feedback ----------------------------------
_q1ef = _decl("mqo_quantize_1bit_ef", _int, _vp, _vp, _u64, _u64, _vp, _vp, _int)


def quantize_1bit_ef(grad, residual, bucket, dtype="f32"):
    """Returns (codes, ranges, new residual); `residual` itself is not modified."""
    grad = _c(grad, np.uint16 if dtype == "bf16" else np.float32)
    n = grad.size
    res = np.array(residual, np.float32, copy=True)
    assert res.size == n
    codes = np.zeros(code_words(n, 1), np.uint32)
    ranges = np.zeros(2 * num_buckets(n, bucket) if n else 0, np.float32)
    rc = _q1ef(_ptr(grad), _ptr(res), n, bucket, _ptr(codes), _ptr(ranges), 1 if dtype == "bf16" else 0)
    if rc:
        raise ValueError("mqo_quantize_1bit_ef failed: %d" % rc)
    return codes, ranges, res
