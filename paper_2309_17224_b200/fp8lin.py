"""Python face of ``libfp8lin.so``: argument marshalling only.

Every function here has the name and the argument order of the C entry point
declared in ``include/fp8lin.h``; tensors are torch CUDA tensors whose
``data_ptr()`` is handed through, the stream is torch's current stream.  There
is no arithmetic and no fallback in this module: if the library is missing the
import fails, and a non-zero status raises ``Fp8Error``.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_int, c_int32, c_int64, c_uint, c_uint64, c_void_p, c_float, c_char_p, POINTER, byref

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfp8lin.so")

OK = 0
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_DTYPE, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_TOO_LARGE = range(1, 9)
E4, E5 = 0, 1
CONV_PAPER, CONV_NATIVE = 0, 1
BF16, F16, F32 = 0, 1, 2
GROUP_AMAX_CAST, GROUP_PREDICTED, GROUP_AMAX_ONLY, GROUP_CAST_ONLY = 0, 1, 2, 3
MM_FWD, MM_DGRAD, MM_WGRAD = 0, 1, 2
ACT_NONE = 0
ACT_GELU = 1
ACT_SWIGLU = 2
FLAG_NONFINITE_AMAX, FLAG_ZERO_AMAX, FLAG_SATURATED, FLAG_TIMEOUT = 1, 2, 4, 8

SYMBOLS = (
    "fp8_create", "fp8_destroy", "fp8_status_string", "fp8_device_flags", "fp8_amax", "fp8_scaling_bias",
    "fp8_scaling_bias_host", "fp8_cast_e4", "fp8_cast_e5", "fp8_ptq_weights", "fp8_linear_fwd", "fp8_linear_dgrad",
    "fp8_linear_wgrad", "fp8_amax_noalloc", "fp8_linear_fwd_act", "fp8_cast_predicted", "fp8_prediction_stats",
    "fp8_linear_dgrad_act", "fp8_selftest_wait_expiry", "fp8_range_stats", "fp8_linear_fwd_q", "fp8_linear_dgrad_q", "fp8_amax_history_bias", "fp8_launch_count", "fp8_cast_group", "fp8_selftest_mma_ceiling", "fp8_bias_log_append", "fp8_bias_mode", "fp8_linear_f16acc", "fp8_linear_infer", "fp8_linear_infer_cast", "fp8_linear_group",
    "fp8h_gelu", "fp8h_gelu_backward", "fp8h_mse_grad", "fp8h_sgd",
)

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2309_17224_b200.build` "
        "(there is no fallback implementation)")

_lib = ctypes.CDLL(LIB_PATH)

_P = c_void_p
_lib.fp8_create.argtypes = [POINTER(c_void_p), c_int]
_lib.fp8_destroy.argtypes = [_P]
_lib.fp8_status_string.argtypes = [c_int]
_lib.fp8_status_string.restype = c_char_p
_lib.fp8_device_flags.argtypes = [_P, _P, POINTER(c_uint), c_int]
_lib.fp8_selftest_wait_expiry.argtypes = [_P, ctypes.c_uint64, _P]
_lib.fp8_selftest_mma_ceiling.argtypes = [_P, _P, _P, c_int64, c_int64, c_int64, _P]
_lib.fp8_bias_log_append.argtypes = [_P, _P, c_int32, _P, c_int32, c_int32, _P, _P, c_int32, _P]
_lib.fp8_bias_mode.argtypes = [_P, _P, c_int32, _P, c_int32, c_int32, c_int32, _P, _P, _P, _P]
_lib.fp8_amax.argtypes = [_P, _P, c_int, c_int64, c_int64, c_int64, _P, _P]
_lib.fp8_amax_noalloc.argtypes = [_P, c_int, c_int64, c_int64, c_int64, _P, _P]
_lib.fp8_scaling_bias.argtypes = [_P, _P, c_int, c_int, c_int32, _P, _P]
_lib.fp8_scaling_bias_host.argtypes = [c_float, c_int, c_int, c_int32, POINTER(c_int32)]
_cast_args = [_P, _P, c_int, c_int64, c_int64, c_int64, _P, c_int, c_int32, _P, _P, _P, _P, _P]
_lib.fp8_cast_e4.argtypes = _cast_args
_lib.fp8_cast_e5.argtypes = _cast_args
_lib.fp8_cast_predicted.argtypes = [_P, c_int, _P, c_int, c_int64, c_int64, c_int64, c_int, c_int32, _P, _P, _P, _P]
_lib.fp8_prediction_stats.argtypes = [_P, _P, POINTER(c_uint), POINTER(c_uint), c_int]
_lib.fp8_range_stats.argtypes = [_P, c_int, _P, c_int, c_int64, c_int64, c_int64, _P, c_int, _P, _P]
_lib.fp8_ptq_weights.argtypes = [_P, _P, c_int, c_int64, c_int64, c_int64, c_int, _P, _P, _P, _P, _P]
_lib.fp8_linear_fwd.argtypes = [_P, _P, _P, _P, _P, _P, c_int, _P, c_int, _P, c_int64, c_int64, c_int64, c_int, _P]
_lib.fp8_linear_infer.argtypes = _lib.fp8_linear_fwd.argtypes
_lib.fp8_linear_infer_cast.argtypes = [_P, _P, c_int, c_int, _P, _P, _P, _P, _P, _P, c_int, _P, c_int, _P, c_int64, c_int64,
                                       c_int64, c_int, _P]
_lib.fp8_linear_fwd_act.argtypes = [_P, _P, _P, _P, _P, _P, c_int, _P, _P, c_int, _P, c_int64, c_int64, c_int64, c_int, _P]
_lib.fp8_linear_dgrad.argtypes = [_P, _P, _P, _P, _P, _P, _P, c_int, _P, c_int64, c_int64, c_int64, c_int, _P]
_lib.fp8_linear_dgrad_act.argtypes = [_P, _P, _P, _P, _P, _P, _P, _P, _P, c_int, _P, c_int64, c_int64, c_int64, c_int, _P]
_lib.fp8_amax_history_bias.argtypes = [_P, _P, c_int32, _P, _P, c_int, c_int, c_int32, _P, _P]
_lib.fp8_linear_fwd_q.argtypes = [_P, _P, _P, _P, _P, _P, c_int, c_int, _P, _P, _P, _P, _P, c_int64, c_int64, c_int64,
                                  c_int, _P]
_lib.fp8_linear_dgrad_q.argtypes = [_P, _P, _P, _P, _P, _P, c_int, _P, _P, _P, _P, _P, _P, c_int64, c_int64, c_int64,
                                    c_int, _P]
_lib.fp8_linear_f16acc.argtypes = [_P, c_int, _P, _P, _P, _P, _P, c_int, c_int32, c_int64, c_int64, c_int64, c_int, _P]
_lib.fp8_linear_wgrad.argtypes = [_P, _P, _P, _P, _P, _P, _P, _P, c_int, c_int64, c_int64, c_int64, c_int, _P]


class GroupItem(ctypes.Structure):
    """``fp8_group_item_t``."""
    _fields_ = [("x", c_void_p), ("x_dt", c_int), ("rows", c_int64), ("cols", c_int64), ("ld", c_int64),
                ("fmt", c_int), ("margin", c_int32), ("d_amax", c_void_p), ("d_bias", c_void_p), ("y", c_void_p)]


_lib.fp8_cast_group.argtypes = [_P, POINTER(GroupItem), c_int32, c_int, c_int32, _P]


class MatmulItem(ctypes.Structure):
    """``fp8_matmul_item_t``."""
    _fields_ = [("kind", c_int32), ("bias_dt", c_int32), ("a8", c_void_p), ("d_ba", c_void_p), ("b8", c_void_p),
                ("d_bb", c_void_p), ("bias_vec", c_void_p), ("out", c_void_p), ("d_amax_out", c_void_p),
                ("out_dt", c_int32), ("reserved", c_int32), ("T", c_int64), ("K", c_int64), ("N", c_int64)]


_lib.fp8_linear_group.argtypes = [_P, POINTER(MatmulItem), c_int32, c_int, _P]
_lib.fp8h_gelu.argtypes = [_P, _P, c_int64, _P]
_lib.fp8h_gelu_backward.argtypes = [_P, _P, _P, c_int64, _P]
_lib.fp8h_mse_grad.argtypes = [_P, _P, ctypes.c_float, _P, c_int64, _P]
_lib.fp8h_sgd.argtypes = [_P, _P, ctypes.c_float, _P, c_int64, _P]
for _name in SYMBOLS:
    if _name != "fp8_status_string":
        getattr(_lib, _name).restype = c_int


class Fp8Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def status_string(status: int) -> str:
    return _lib.fp8_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise Fp8Error(status, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


_DT = {torch.bfloat16: BF16, torch.float16: F16, torch.float32: F32}


def _ld(x):
    """Leading dimension of a 2-D tensor (torch leaves the stride of a size-1 dimension arbitrary)."""
    return x.stride(0) if x.shape[0] > 1 else x.shape[1]


def launch_count() -> int:
    """Kernels this library has launched in this process so far."""
    out = c_uint64(0)
    _check(_lib.fp8_launch_count(byref(out)), "fp8_launch_count")
    return out.value


def scaling_bias_host(amax: float, fmt: int, conv: int = CONV_PAPER, margin: int = 0) -> int:
    out = c_int32(0)
    _check(_lib.fp8_scaling_bias_host(c_float(amax), fmt, conv, margin, byref(out)), "fp8_scaling_bias_host")
    return out.value


def amax_noalloc(x, d_amax, rows=None, cols=None, ld=None):
    """``fp8_amax_noalloc``: amax without a context and without any device
    allocation by the library (for callers that own all device memory or may
    not call cudaMalloc).  Contiguous bf16 input of at most 2^29 elements;
    calls on one device must not overlap on the GPU."""
    rows = x.shape[0] if rows is None else rows
    cols = x.shape[1] if cols is None else cols
    ld = _ld(x) if ld is None else ld
    _check(_lib.fp8_amax_noalloc(_ptr(x), _DT[x.dtype], rows, cols, ld, _ptr(d_amax), _stream()), "fp8_amax_noalloc")


def group_items(tensors):
    """A ctypes array of ``fp8_group_item_t`` from (fmt, x, d_amax, d_bias, y[, margin]) tuples; build it once
    and hand it to ``Context.cast_group`` every step (the tensors must stay alive)."""
    arr = (GroupItem * len(tensors))()
    for it, t in zip(arr, tensors):
        fmt, x, d_amax, d_bias, y = t[:5]
        it.x, it.x_dt, it.rows, it.cols, it.ld = x.data_ptr(), _DT[x.dtype], x.shape[0], x.shape[1], _ld(x)
        it.fmt, it.margin = fmt, (t[5] if len(t) > 5 else 0)
        it.d_amax = d_amax.data_ptr() if d_amax is not None else None
        it.d_bias, it.y = d_bias.data_ptr(), (y.data_ptr() if y is not None else None)
    return arr


MATMUL_FWD, MATMUL_DGRAD, MATMUL_WGRAD = 0, 1, 2


def matmul_items(matmuls):
    """A ctypes array of ``fp8_matmul_item_t`` from (kind, a8, d_ba, b8, d_bb, out[, bias_vec[, d_amax_out]]) tuples
    (row-major operands: FWD x8, w8 -> y; DGRAD dy8, w8 -> dx; WGRAD dy8, x8 -> dw); build it once and hand it to
    ``Context.linear_group`` every step (the tensors must stay alive)."""
    arr = (MatmulItem * len(matmuls))()
    for it, m in zip(arr, matmuls):
        kind, a8, d_ba, b8, d_bb, out = m[:6]
        bias_vec = m[6] if len(m) > 6 else None
        d_amax_out = m[7] if len(m) > 7 else None
        if kind == MATMUL_FWD:
            (T, K), N = a8.shape, b8.shape[0]
        elif kind == MATMUL_DGRAD:
            (T, N), K = a8.shape, b8.shape[1]
        else:
            (T, N), K = a8.shape, b8.shape[1]
        it.kind, it.T, it.K, it.N = kind, T, K, N
        it.a8, it.d_ba, it.b8, it.d_bb = a8.data_ptr(), d_ba.data_ptr(), b8.data_ptr(), d_bb.data_ptr()
        it.bias_vec = bias_vec.data_ptr() if bias_vec is not None else None
        it.bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        it.out, it.out_dt = out.data_ptr(), _DT[out.dtype]
        it.d_amax_out = d_amax_out.data_ptr() if d_amax_out is not None else None
    return arr


# -- element-wise kernels of the stress stack (include/fp8_harness.h): harness, not the paper's method -----------------
def _bf16(t):
    assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.is_cuda, "contiguous bf16 CUDA tensor expected"
    return t


def harness_gelu(x, y):
    _check(_lib.fp8h_gelu(_ptr(_bf16(x)), _ptr(_bf16(y)), x.numel(), _stream()), "fp8h_gelu")


def harness_gelu_backward(g, pre, out):
    _check(_lib.fp8h_gelu_backward(_ptr(_bf16(g)), _ptr(_bf16(pre)), _ptr(_bf16(out)), g.numel(), _stream()), "fp8h_gelu_backward")


def harness_mse_grad(y, target, scale, g):
    _check(_lib.fp8h_mse_grad(_ptr(_bf16(y)), _ptr(_bf16(target)), float(scale), _ptr(_bf16(g)), y.numel(), _stream()),
           "fp8h_mse_grad")


def harness_sgd(w32, dw, lr, w16):
    assert w32.dtype == torch.float32 and w32.is_contiguous()
    _check(_lib.fp8h_sgd(_ptr(w32), _ptr(_bf16(dw)), float(lr), _ptr(_bf16(w16)), w32.numel(), _stream()), "fp8h_sgd")


class Context:
    """Owns one ``fp8_ctx``.  All methods launch on torch's current stream."""

    def __init__(self, device: int = 0):
        self._h = c_void_p()
        self.device = device
        _check(_lib.fp8_create(byref(self._h), device), "fp8_create")

    def close(self):
        if self._h:
            _lib.fp8_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- status ---------------------------------------------------------------
    def device_flags(self, clear: bool = True) -> int:
        flags = c_uint(0)
        st = _lib.fp8_device_flags(self._h, _stream(), byref(flags), 1 if clear else 0)
        if st not in (OK, ERR_DEVICE_TIMEOUT):
            _check(st, "fp8_device_flags")
        return flags.value

    def selftest_wait_expiry(self, limit_ns: int = 1_000_000):
        """Make one bounded device-side wait run out on purpose (raises FP8_FLAG_TIMEOUT, no fault)."""
        _check(_lib.fp8_selftest_wait_expiry(self._h, ctypes.c_uint64(limit_ns), _stream()), "fp8_selftest_wait_expiry")

    def selftest_mma_ceiling(self, out, d_zero, K: int):
        """The CTA-pair matmul kernel on an out.shape[0] x out.shape[1] x K problem with its operand loads off."""
        _check(_lib.fp8_selftest_mma_ceiling(self._h, _ptr(out), _ptr(d_zero), out.shape[0], out.shape[1], K, _stream()),
               "fp8_selftest_mma_ceiling")

    # -- amax / bias ------------------------------------------------------------
    def amax(self, x, d_amax, rows=None, cols=None, ld=None):
        rows = x.shape[0] if rows is None else rows
        cols = x.shape[1] if cols is None else cols
        ld = _ld(x) if ld is None else ld
        _check(_lib.fp8_amax(self._h, _ptr(x), _DT[x.dtype], rows, cols, ld, _ptr(d_amax), _stream()), "fp8_amax")

    def scaling_bias(self, d_amax, fmt, conv, margin, d_bias):
        _check(_lib.fp8_scaling_bias(self._h, _ptr(d_amax), fmt, conv, margin, _ptr(d_bias), _stream()),
               "fp8_scaling_bias")

    def amax_history_bias(self, d_history, d_cursor, d_amax_new, fmt, d_bias, conv=CONV_PAPER, margin=0):
        _check(_lib.fp8_amax_history_bias(self._h, _ptr(d_history), d_history.numel(), _ptr(d_cursor), _ptr(d_amax_new),
                                          fmt, conv, margin, _ptr(d_bias), _stream()), "fp8_amax_history_bias")

    # -- bias log ---------------------------------------------------------------
    def bias_log_append(self, d_ring, d_head, step, first_tensor_id, d_amax, d_bias):
        """``fp8_bias_log_append``: d_ring is an int32 tensor [capacity, 4] (one ``fp8_bias_record_t`` per row: step,
        tensor id, amax bits, bias), d_head an int64 scalar tensor; d_amax / d_bias are 1-D device arrays."""
        _check(_lib.fp8_bias_log_append(self._h, _ptr(d_ring), d_ring.shape[0], _ptr(d_head), step, first_tensor_id,
                                        _ptr(d_amax), _ptr(d_bias), d_amax.numel(), _stream()), "fp8_bias_log_append")

    def bias_mode(self, d_ring, d_head, tensor_id, step_lo, step_hi, d_mode, d_count, d_samples=None):
        _check(_lib.fp8_bias_mode(self._h, _ptr(d_ring), d_ring.shape[0], _ptr(d_head), tensor_id, step_lo, step_hi,
                                  _ptr(d_mode), _ptr(d_count), _ptr(d_samples), _stream()), "fp8_bias_mode")

    # -- cast -------------------------------------------------------------------
    def _cast(self, fn, name, x, d_bias, conv, margin, d_amax_out, d_bias_out, y, y_t, rows, cols, ld):
        rows = x.shape[0] if rows is None else rows
        cols = x.shape[1] if cols is None else cols
        ld = _ld(x) if ld is None else ld
        _check(fn(self._h, _ptr(x), _DT[x.dtype], rows, cols, ld, _ptr(d_bias), conv, margin, _ptr(d_amax_out),
                  _ptr(d_bias_out), _ptr(y), _ptr(y_t), _stream()), name)

    def cast_e4(self, x, d_bias, conv=CONV_PAPER, margin=0, d_amax_out=None, d_bias_out=None, y=None, y_t=None,
                rows=None, cols=None, ld=None):
        self._cast(_lib.fp8_cast_e4, "fp8_cast_e4", x, d_bias, conv, margin, d_amax_out, d_bias_out, y, y_t, rows,
                   cols, ld)

    def cast_e5(self, x, d_bias, conv=CONV_PAPER, margin=0, d_amax_out=None, d_bias_out=None, y=None, y_t=None,
                rows=None, cols=None, ld=None):
        self._cast(_lib.fp8_cast_e5, "fp8_cast_e5", x, d_bias, conv, margin, d_amax_out, d_bias_out, y, y_t, rows,
                   cols, ld)

    def cast_predicted(self, fmt, x, d_amax_out, d_bias_inout, y, conv=CONV_PAPER, margin=0, rows=None, cols=None,
                       ld=None):
        rows = x.shape[0] if rows is None else rows
        cols = x.shape[1] if cols is None else cols
        ld = _ld(x) if ld is None else ld
        _check(_lib.fp8_cast_predicted(self._h, fmt, _ptr(x), _DT[x.dtype], rows, cols, ld, conv, margin,
                                       _ptr(d_amax_out), _ptr(d_bias_inout), _ptr(y), _stream()), "fp8_cast_predicted")

    def cast_group(self, items, conv=CONV_PAPER, predicted=False, mode=None):
        """``fp8_cast_group``.  `items`: a ``group_items(...)`` array, or a list of (fmt, x, d_amax, d_bias, y[, margin])
        tuples that is marshalled on the spot.  `mode`: one of the GROUP_* constants (default: GROUP_PREDICTED if
        `predicted` else GROUP_AMAX_CAST)."""
        arr = items if isinstance(items, ctypes.Array) else group_items(items)
        if mode is None:
            mode = GROUP_PREDICTED if predicted else GROUP_AMAX_CAST
        _check(_lib.fp8_cast_group(self._h, arr, len(arr), conv, mode, _stream()), "fp8_cast_group")

    def prediction_stats(self, clear: bool = True):
        hits, misses = c_uint(0), c_uint(0)
        _check(_lib.fp8_prediction_stats(self._h, _stream(), byref(hits), byref(misses), 1 if clear else 0),
               "fp8_prediction_stats")
        return hits.value, misses.value

    def range_stats(self, fmt, x, d_bias, d_counts, conv=CONV_PAPER, rows=None, cols=None, ld=None):
        """d_counts: 4 x int64 on the device = clipped, flushed to zero, subnormal, non-zero finite."""
        rows = x.shape[0] if rows is None else rows
        cols = x.shape[1] if cols is None else cols
        ld = _ld(x) if ld is None else ld
        _check(_lib.fp8_range_stats(self._h, fmt, _ptr(x), _DT[x.dtype], rows, cols, ld, _ptr(d_bias), conv,
                                    _ptr(d_counts), _stream()), "fp8_range_stats")

    def ptq_weights(self, w, conv, w8, w8_t, d_bw, d_amax_w):
        _check(_lib.fp8_ptq_weights(self._h, _ptr(w), _DT[w.dtype], w.shape[0], w.shape[1], _ld(w), conv,
                                    _ptr(w8), _ptr(w8_t), _ptr(d_bw), _ptr(d_amax_w), _stream()), "fp8_ptq_weights")

    # -- matmuls ----------------------------------------------------------------
    def linear_fwd(self, x8, d_bx, w8, d_bw, y, bias_vec=None, d_amax_y=None, conv=CONV_PAPER):
        T, K = x8.shape
        N = w8.shape[0]
        bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        _check(_lib.fp8_linear_fwd(self._h, _ptr(x8), _ptr(d_bx), _ptr(w8), _ptr(d_bw), _ptr(bias_vec), bias_dt,
                                   _ptr(y), _DT[y.dtype], _ptr(d_amax_y), T, K, N, conv, _stream()),
               "fp8_linear_fwd")

    def linear_infer(self, x8, d_bx, w8, d_bw, y, bias_vec=None, d_amax_y=None, conv=CONV_PAPER):
        """``fp8_linear_infer``: linear_fwd for weights whose bytes were final before the launch ahead of this call."""
        T, K = x8.shape
        N = w8.shape[0]
        bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        _check(_lib.fp8_linear_infer(self._h, _ptr(x8), _ptr(d_bx), _ptr(w8), _ptr(d_bw), _ptr(bias_vec), bias_dt,
                                     _ptr(y), _DT[y.dtype], _ptr(d_amax_y), T, K, N, conv, _stream()),
               "fp8_linear_infer")

    def linear_infer_cast(self, x, d_amax_x, d_bx, x8, w8, d_bw, y, margin=0, bias_vec=None, d_amax_y=None, conv=CONV_PAPER):
        """``fp8_linear_infer_cast``: FP8-AMAX of the activation x and the forward matmul on weights quantised once."""
        T, K = x.shape
        N = w8.shape[0]
        bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        _check(_lib.fp8_linear_infer_cast(self._h, _ptr(x), _DT[x.dtype], margin, _ptr(d_amax_x), _ptr(d_bx), _ptr(x8),
                                          _ptr(w8), _ptr(d_bw), _ptr(bias_vec), bias_dt, _ptr(y), _DT[y.dtype],
                                          _ptr(d_amax_y), T, K, N, conv, _stream()), "fp8_linear_infer_cast")

    def linear_group(self, items, conv=CONV_PAPER):
        """``fp8_linear_group``: independent matmuls in one launch.  `items`: a ``matmul_items(...)`` array or the list
        of tuples it is built from."""
        arr = items if isinstance(items, ctypes.Array) else matmul_items(items)
        _check(_lib.fp8_linear_group(self._h, arr, len(arr), conv, _stream()), "fp8_linear_group")

    def linear_fwd_act(self, x8, d_bx, w8, d_bw, y_pre, y_act, bias_vec=None, d_amax_act=None, act=ACT_GELU,
                       conv=CONV_PAPER):
        T, K = x8.shape
        N = w8.shape[0]
        bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        _check(_lib.fp8_linear_fwd_act(self._h, _ptr(x8), _ptr(d_bx), _ptr(w8), _ptr(d_bw), _ptr(bias_vec), bias_dt,
                                       _ptr(y_pre), _ptr(y_act), act, _ptr(d_amax_act), T, K, N, conv, _stream()),
               "fp8_linear_fwd_act")

    def linear_dgrad(self, dy8, d_bg, w8, w8_t, d_bw, dx, d_amax_dx=None, conv=CONV_PAPER):
        T, N = dy8.shape
        K = dx.shape[1]
        _check(_lib.fp8_linear_dgrad(self._h, _ptr(dy8), _ptr(d_bg), _ptr(w8), _ptr(w8_t), _ptr(d_bw), _ptr(dx),
                                     _DT[dx.dtype], _ptr(d_amax_dx), T, K, N, conv, _stream()), "fp8_linear_dgrad")

    def linear_dgrad_act(self, dy8, d_bg, w8, w8_t, d_bw, y_pre, dx, dx_act, d_amax_act=None, act=ACT_GELU,
                         conv=CONV_PAPER):
        T, N = dy8.shape
        K = w8.shape[1] if w8 is not None else w8_t.shape[0]
        _check(_lib.fp8_linear_dgrad_act(self._h, _ptr(dy8), _ptr(d_bg), _ptr(w8), _ptr(w8_t), _ptr(d_bw), _ptr(y_pre),
                                         _ptr(dx), _ptr(dx_act), act, _ptr(d_amax_act), T, K, N, conv, _stream()),
               "fp8_linear_dgrad_act")

    def linear_fwd_q(self, x8, d_bx, w8, d_bw, z8, d_bz, y_pre=None, z=None, bias_vec=None, d_amax_z=None,
                     act=ACT_NONE, conv=CONV_PAPER):
        T, K = x8.shape
        N = w8.shape[0]
        bias_dt = _DT[bias_vec.dtype] if bias_vec is not None else BF16
        _check(_lib.fp8_linear_fwd_q(self._h, _ptr(x8), _ptr(d_bx), _ptr(w8), _ptr(d_bw), _ptr(bias_vec), bias_dt, act,
                                     _ptr(y_pre), _ptr(z), _ptr(z8), _ptr(d_bz), _ptr(d_amax_z), T, K, N, conv,
                                     _stream()), "fp8_linear_fwd_q")

    def linear_dgrad_q(self, dy8, d_bg, w8, w8_t, d_bw, g8, d_bq, y_pre=None, dx=None, g=None, d_amax_g=None,
                       act=ACT_NONE, conv=CONV_PAPER):
        T, N = dy8.shape
        K = w8.shape[1] if w8 is not None else w8_t.shape[0]
        _check(_lib.fp8_linear_dgrad_q(self._h, _ptr(dy8), _ptr(d_bg), _ptr(w8), _ptr(w8_t), _ptr(d_bw), act,
                                       _ptr(y_pre), _ptr(dx), _ptr(g), _ptr(g8), _ptr(d_bq), _ptr(d_amax_g), T, K, N,
                                       conv, _stream()), "fp8_linear_dgrad_q")

    def linear_f16acc(self, kind, a8, d_ba, b8, d_bb, out, T, K, N, chunk=128, conv=CONV_PAPER):
        """``fp8_linear_f16acc``: the matmul of `kind` with FP16 accumulation emulated; out is float16 or float32."""
        _check(_lib.fp8_linear_f16acc(self._h, kind, _ptr(a8), _ptr(d_ba), _ptr(b8), _ptr(d_bb), _ptr(out), _DT[out.dtype],
                                      chunk, T, K, N, conv, _stream()), "fp8_linear_f16acc")

    def linear_wgrad(self, dy8, dy8_t, d_bg, x8, x8_t, d_bx, dw, T, conv=CONV_PAPER):
        N, K = dw.shape
        _check(_lib.fp8_linear_wgrad(self._h, _ptr(dy8), _ptr(dy8_t), _ptr(d_bg), _ptr(x8), _ptr(x8_t), _ptr(d_bx),
                                     _ptr(dw), _DT[dw.dtype], T, K, N, conv, _stream()), "fp8_linear_wgrad")


def raw():
    """The ctypes library handle (for tests of the C ABI itself)."""
    return _lib
