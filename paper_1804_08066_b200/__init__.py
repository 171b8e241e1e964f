"""libmqgrad for B200: Python binding of the C ABI in include/mqgrad.h.

The binding only marshals arguments: torch CUDA tensors supply the device pointers and the
current torch stream supplies the CUDA stream; every step of the path runs in the CUDA
kernels of libmqgrad.so.  There is no CPU fallback: a missing library or a CPU tensor
raises.

Function names and argument order follow the C ABI:
  mqg_quantize, mqg_quantize_workers, mqg_dequant_accumulate, mqg_apply, mqg_server_step,
  mqg_server_requantize, mqg_quantize_segments, mqg_quantize_segments_workers, mqg_server_step_segments, mqg_quantize_minmax,
  mqg_quantize_workers_minmax,
  mqg_dequant_accumulate_minmax, mqg_server_step_minmax, mqg_quantize_l2, mqg_quantize_workers_l2, mqg_quantize_segments_l2,
  mqg_l2_workspace_floats, mqg_quantize_segments_l2_static, mqg_quantize_1bit_ef, mqg_code_words, mqg_num_buckets,
  mqg_wire_bytes, mqg_last_error, mqg_version, mqg_device_timeouts, mqg_check_timeouts,
  mqg_test_wait_override.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmqgrad.so")

MQG_OK = 0
MQG_ERR_INVALID = -1
MQG_ERR_BITS = -2
MQG_ERR_ALIGN = -3
MQG_ERR_TOO_MANY_WORKERS = -4
MQG_ERR_CUDA = -5
MQG_ERR_TIMEOUT = -6
MQG_F32, MQG_BF16 = 0, 1
MQG_MAX_WORKERS = 32


class MqgError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("libmqgrad status %d: %s" % (status, message))
        self.status = status


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libmqgrad.so is not built (%s); run `python paper_1804_08066_b200/build.py`. "
            "There is no fallback path." % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    u64, u32, i32, vp, f32 = C.c_uint64, C.c_uint32, C.c_int, C.c_void_p, C.c_float
    sigs = {
        "mqg_code_words": (C.c_size_t, [u64, i32]),
        "mqg_num_buckets": (C.c_size_t, [u64, u64]),
        "mqg_wire_bytes": (C.c_size_t, [u64, i32, u64]),
        "mqg_last_error": (C.c_char_p, []),
        "mqg_version": (i32, []),
        "mqg_device_timeouts": (i32, [C.POINTER(C.c_uint)]),
        "mqg_check_timeouts": (i32, [C.POINTER(C.c_uint), i32]),
        "mqg_test_wait_override": (i32, [u32, i32]),
        "mqg_quantize": (i32, [vp, u64, i32, u64, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_quantize_workers": (i32, [vp, i32, u64, i32, u64, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_dequant_accumulate": (i32, [vp, vp, i32, i32, u64, vp, u64, i32, vp]),
        "mqg_apply": (i32, [vp, vp, f32, u64, vp]),
        "mqg_quantize_minmax": (i32, [vp, u64, i32, u64, vp, vp, i32, vp]),
        "mqg_quantize_workers_minmax": (i32, [vp, i32, u64, i32, u64, vp, vp, i32, vp]),
        "mqg_dequant_accumulate_minmax": (i32, [vp, vp, i32, i32, u64, vp, u64, i32, vp]),
        "mqg_server_step_minmax": (i32, [vp, vp, i32, i32, u64, u64, vp, f32, vp, vp]),
        "mqg_server_step": (i32, [vp, vp, i32, i32, u64, u64, vp, f32, vp, vp]),
        "mqg_server_requantize": (i32, [vp, vp, i32, i32, u64, u64, f32, u64, vp, vp, u32, u32, vp]),
        "mqg_quantize_segments": (i32, [vp, i32, vp, vp, i32, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_server_step_segments": (i32, [vp, vp, i32, i32, i32, vp, vp, vp, f32, vp, vp]),
        "mqg_quantize_segments_workers": (i32, [vp, i32, i32, vp, vp, i32, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_quantize_1bit_ef": (i32, [vp, vp, u64, u64, vp, vp, i32, vp]),
        "mqg_quantize_l2": (i32, [vp, u64, i32, u64, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_quantize_workers_l2": (i32, [vp, i32, u64, i32, u64, u64, vp, vp, i32, u32, u32, u64, vp]),
        "mqg_l2_workspace_floats": (C.c_size_t, [i32, vp]),
        "mqg_quantize_segments_l2": (i32, [vp, i32, vp, vp, i32, u64, vp, vp, i32, u32, u32, u64, vp,
                                           C.c_size_t, vp]),
        "mqg_quantize_segments_l2_static": (i32, [vp, i32, vp, vp, i32, u64, vp, vp, i32, u32, u32, u64, vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


class _LazyLibrary:
    """Loads libmqgrad.so at the first call instead of at import, so that a process which only
    imports the input generators (workloads.py) never maps the library."""

    def __init__(self):
        self._lib = None

    def __getattr__(self, name):
        if self._lib is None:
            self._lib = _load()
        return getattr(self._lib, name)


_lib = _LazyLibrary()


def _check(status: int) -> None:
    if status != MQG_OK:
        raise MqgError(status, _lib.mqg_last_error().decode())


def _dev_ptr(t, what: str) -> int:
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor (libmqgrad has no CPU path)" % what)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % what)
    return t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _ptr_table(tensors, what: str):
    return (C.c_void_p * len(tensors))(*[_dev_ptr(t, "%s[%d]" % (what, i))
                                         for i, t in enumerate(tensors)])


def _u64_table(values):
    vals = [int(v) for v in values]
    return (C.c_uint64 * len(vals))(*vals)


def mqg_code_words(n: int, bits: int) -> int:
    return int(_lib.mqg_code_words(n, bits))


def mqg_num_buckets(n: int, bucket: int) -> int:
    return int(_lib.mqg_num_buckets(n, bucket))


def mqg_wire_bytes(n: int, bits: int, bucket: int) -> int:
    return int(_lib.mqg_wire_bytes(n, bits, bucket))


def mqg_last_error() -> str:
    return _lib.mqg_last_error().decode()


def mqg_version() -> int:
    return int(_lib.mqg_version())


def mqg_device_timeouts() -> int:
    """Number of kernel waits that gave up on the current device (synchronises); 0 when healthy."""
    c = C.c_uint(0)
    _check(_lib.mqg_device_timeouts(C.byref(c)))
    return int(c.value)


def mqg_check_timeouts(reset: bool = True) -> int:
    """Waits that ran out on the current device since the last reset (synchronises).  Raises MqgError
    with status MQG_ERR_TIMEOUT when there were any, after clearing the counter if `reset`; returns 0
    otherwise."""
    c = C.c_uint(0)
    _check(_lib.mqg_check_timeouts(C.byref(c), 1 if reset else 0))
    return int(c.value)


def mqg_test_wait_override(poll_limit: int = 0, arm_only: bool = False) -> None:
    """Test hook of the C ABI (see include/mqgrad.h); (0, False) restores normal operation."""
    _check(_lib.mqg_test_wait_override(poll_limit, 1 if arm_only else 0))


def _grad_dtype(grad) -> int:
    import torch
    if grad.dtype == torch.float32:
        return MQG_F32
    if grad.dtype == torch.bfloat16:
        return MQG_BF16
    raise TypeError("grad must be float32 or bfloat16, got %s" % grad.dtype)


def mqg_quantize(grad, n: int, bits: int, bucket: int, seed: int, codes, scales,
                 worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    """Quantize(g, K): writes `codes` (uint32/int32 words) and `scales` (float32)."""
    _check(_lib.mqg_quantize(_dev_ptr(grad, "grad") if n else None, n, bits, bucket,
                             seed & 0xFFFFFFFFFFFFFFFF,
                             _dev_ptr(codes, "codes") if n else None,
                             _dev_ptr(scales, "scales") if n else None,
                             _grad_dtype(grad), worker, step, elem_offset, _stream()))


def mqg_quantize_workers(grads, W: int, n: int, bits: int, bucket: int, seed: int, codes, scales,
                         first_worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    """Quantize(g_p, K) for W workers' gradients (lists of W tensors) in one launch."""
    if len(grads) != W or len(codes) != W or len(scales) != W:
        raise ValueError("grads, codes and scales must each hold W tensors")
    dtypes = {_grad_dtype(g) for g in grads}
    if len(dtypes) != 1:
        raise TypeError("all gradients must have the same dtype")
    _check(_lib.mqg_quantize_workers(_ptr_table(grads, "grads"), W, n, bits, bucket,
                                     seed & 0xFFFFFFFFFFFFFFFF, _ptr_table(codes, "codes"),
                                     _ptr_table(scales, "scales"), dtypes.pop(), first_worker, step,
                                     elem_offset, _stream()))


def mqg_quantize_workers_l2(grads, W: int, n: int, bits: int, bucket: int, seed: int, codes, scales,
                            first_worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    """The L2-norm scale variant for W workers' gradients (lists of W tensors) in one launch."""
    if len(grads) != W or len(codes) != W or len(scales) != W:
        raise ValueError("grads, codes and scales must each hold W tensors")
    dtypes = {_grad_dtype(g) for g in grads}
    if len(dtypes) != 1:
        raise TypeError("all gradients must have the same dtype")
    _check(_lib.mqg_quantize_workers_l2(_ptr_table(grads, "grads"), W, n, bits, bucket,
                                        seed & 0xFFFFFFFFFFFFFFFF, _ptr_table(codes, "codes"),
                                        _ptr_table(scales, "scales"), dtypes.pop(), first_worker, step,
                                        elem_offset, _stream()))


def mqg_dequant_accumulate(codes, scales, W: int, bits: int, n: int, acc, bucket: int,
                           add_into_acc: bool = False) -> None:
    _check(_lib.mqg_dequant_accumulate(_ptr_table(codes, "codes"), _ptr_table(scales, "scales"),
                                       W, bits, n, _dev_ptr(acc, "acc") if n else None, bucket,
                                       1 if add_into_acc else 0, _stream()))


def mqg_apply(params, acc, lr: float, n: int) -> None:
    _check(_lib.mqg_apply(_dev_ptr(params, "params") if n else None,
                          _dev_ptr(acc, "acc") if n else None, lr, n, _stream()))


def mqg_server_step(codes, scales, W: int, bits: int, n: int, bucket: int, params, lr: float,
                    acc_out=None) -> None:
    _check(_lib.mqg_server_step(_ptr_table(codes, "codes"), _ptr_table(scales, "scales"), W, bits,
                                n, bucket, _dev_ptr(params, "params") if n else None, lr,
                                _dev_ptr(acc_out, "acc_out") if acc_out is not None else None,
                                _stream()))


def mqg_quantize_workers_minmax(grads, W: int, n: int, bits: int, bucket: int, codes, ranges) -> None:
    """The (min, max) variant for W workers' gradients (lists of W tensors) in one launch."""
    if len(grads) != W or len(codes) != W or len(ranges) != W:
        raise ValueError("grads, codes and ranges must each hold W tensors")
    dtypes = {_grad_dtype(g) for g in grads}
    if len(dtypes) != 1:
        raise TypeError("all gradients must have the same dtype")
    _check(_lib.mqg_quantize_workers_minmax(_ptr_table(grads, "grads"), W, n, bits, bucket,
                                            _ptr_table(codes, "codes"), _ptr_table(ranges, "ranges"),
                                            dtypes.pop(), _stream()))


def mqg_quantize_minmax(grad, n: int, bits: int, bucket: int, codes, ranges) -> None:
    """(min, max) nearest-rounding variant: writes `codes` and `ranges` (lo, hi per bucket)."""
    _check(_lib.mqg_quantize_minmax(_dev_ptr(grad, "grad") if n else None, n, bits, bucket,
                                    _dev_ptr(codes, "codes") if n else None,
                                    _dev_ptr(ranges, "ranges") if n else None, _grad_dtype(grad), _stream()))


def mqg_dequant_accumulate_minmax(codes, ranges, W: int, bits: int, n: int, acc, bucket: int,
                                  add_into_acc: bool = False) -> None:
    _check(_lib.mqg_dequant_accumulate_minmax(_ptr_table(codes, "codes"), _ptr_table(ranges, "ranges"),
                                              W, bits, n, _dev_ptr(acc, "acc") if n else None, bucket,
                                              1 if add_into_acc else 0, _stream()))


def mqg_server_step_minmax(codes, ranges, W: int, bits: int, n: int, bucket: int, params, lr: float,
                           acc_out=None) -> None:
    _check(_lib.mqg_server_step_minmax(_ptr_table(codes, "codes"), _ptr_table(ranges, "ranges"), W, bits,
                                       n, bucket, _dev_ptr(params, "params") if n else None, lr,
                                       _dev_ptr(acc_out, "acc_out") if acc_out is not None else None,
                                       _stream()))


def mqg_server_requantize(codes, scales, W: int, bits: int, n: int, bucket: int, mean_scale: float,
                          seed: int, codes_out, scales_out, worker: int = 0, step: int = 0) -> None:
    """Downlink: de-quantize + sum + scale to the mean + quantize again, in one pass."""
    _check(_lib.mqg_server_requantize(_ptr_table(codes, "codes"), _ptr_table(scales, "scales"), W, bits,
                                      n, bucket, mean_scale, seed & 0xFFFFFFFFFFFFFFFF,
                                      _dev_ptr(codes_out, "codes_out") if n else None,
                                      _dev_ptr(scales_out, "scales_out") if n else None,
                                      worker, step, _stream()))


def mqg_quantize_segments(grad, seg_off, code_off, bits: int, seed: int, codes, scales,
                          worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    nseg = len(seg_off) - 1
    _check(_lib.mqg_quantize_segments(_dev_ptr(grad, "grad"), nseg, _u64_table(seg_off),
                                      _u64_table(code_off), bits, seed & 0xFFFFFFFFFFFFFFFF,
                                      _dev_ptr(codes, "codes"), _dev_ptr(scales, "scales"),
                                      _grad_dtype(grad), worker, step, elem_offset, _stream()))


def mqg_quantize_segments_workers(grads, W: int, seg_off, code_off, bits: int, seed: int, codes, scales,
                                  first_worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    nseg = len(seg_off) - 1
    _check(_lib.mqg_quantize_segments_workers(_ptr_table(grads, "grads"), W, nseg, _u64_table(seg_off),
                                              _u64_table(code_off), bits, seed & 0xFFFFFFFFFFFFFFFF,
                                              _ptr_table(codes, "codes"), _ptr_table(scales, "scales"),
                                              _grad_dtype(grads[0]), first_worker, step, elem_offset, _stream()))


def mqg_server_step_segments(codes, scales, W: int, bits: int, seg_off, code_off, params,
                             lr: float, acc_out=None) -> None:
    nseg = len(seg_off) - 1
    _check(_lib.mqg_server_step_segments(_ptr_table(codes, "codes"), _ptr_table(scales, "scales"),
                                         W, bits, nseg, _u64_table(seg_off), _u64_table(code_off),
                                         _dev_ptr(params, "params"), lr,
                                         _dev_ptr(acc_out, "acc_out") if acc_out is not None else None,
                                         _stream()))


def mqg_quantize_1bit_ef(grad, residual, n: int, bucket: int, codes, ranges) -> None:
    """`residual` (float32, n elements) is read and updated in place."""
    _check(_lib.mqg_quantize_1bit_ef(_dev_ptr(grad, "grad"), _dev_ptr(residual, "residual"), n, bucket,
                                     _dev_ptr(codes, "codes"), _dev_ptr(ranges, "ranges"),
                                     _grad_dtype(grad), _stream()))


def mqg_quantize_l2(grad, n: int, bits: int, bucket: int, seed: int, codes, scales,
                    worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    _check(_lib.mqg_quantize_l2(_dev_ptr(grad, "grad"), n, bits, bucket, seed & 0xFFFFFFFFFFFFFFFF,
                                _dev_ptr(codes, "codes"), _dev_ptr(scales, "scales"),
                                _grad_dtype(grad), worker, step, elem_offset, _stream()))


def mqg_l2_workspace_floats(seg_off) -> int:
    return int(_lib.mqg_l2_workspace_floats(len(seg_off) - 1, _u64_table(seg_off)))


def mqg_quantize_segments_l2(grad, seg_off, code_off, bits: int, seed: int, codes, scales, workspace,
                             worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    """`workspace`: float32 CUDA tensor of at least mqg_l2_workspace_floats(seg_off) elements."""
    nseg = len(seg_off) - 1
    _check(_lib.mqg_quantize_segments_l2(_dev_ptr(grad, "grad"), nseg, _u64_table(seg_off),
                                         _u64_table(code_off), bits, seed & 0xFFFFFFFFFFFFFFFF,
                                         _dev_ptr(codes, "codes"), _dev_ptr(scales, "scales"),
                                         _grad_dtype(grad), worker, step, elem_offset,
                                         _dev_ptr(workspace, "workspace"), workspace.numel(), _stream()))


MQG_L2_STATIC_WORKSPACE_FLOATS = 65536


def mqg_quantize_segments_l2_static(grad, seg_off, code_off, bits: int, seed: int, codes, scales,
                                    worker: int = 0, step: int = 0, elem_offset: int = 0) -> None:
    """mqg_quantize_segments_l2 for callers that cannot supply a workspace: the partial sums use an
    array inside the library (at most MQG_L2_STATIC_WORKSPACE_FLOATS of them); calls that may
    overlap on the device must be ordered by the caller."""
    nseg = len(seg_off) - 1
    _check(_lib.mqg_quantize_segments_l2_static(_dev_ptr(grad, "grad"), nseg, _u64_table(seg_off),
                                                _u64_table(code_off), bits, seed & 0xFFFFFFFFFFFFFFFF,
                                                _dev_ptr(codes, "codes"), _dev_ptr(scales, "scales"),
                                                _grad_dtype(grad), worker, step, elem_offset, _stream()))


def raw_library() -> C.CDLL:
    """The ctypes handle, for callers that pass raw device pointers themselves."""
    _lib.mqg_version                       # loads the library if this is its first use
    return _lib._lib
