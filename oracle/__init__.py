"""CPU oracle for the FP8 linear layer -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy front end of ``fp8_oracle.c`` (a plain C restatement of the
paper's method, double precision, no CUDA).  Only the tests, the smoke check
and the benchmark's CPU legs may import this package; the product never does,
and this package never imports the product.

Format ids: ``P_E4``/``P_E5`` are the paper's own FP8 formats (Table 7 rows
"(a)": exponent bias 8 / 16, max 240 / 57344, the negative-zero code is NaN);
``N_E4``/``N_E5`` are the rows "(b)" that the tensor cores consume (bias
7 / 15, max 448 / 57344).

Scaling conventions (how a paper-convention bias ``b`` turns into the shift
that produces native bytes):

* ``CONV_PAPER``: Eq. 3 with the paper format's ``max_num`` (240 / 57344);
  shift ``s = b + delta`` with ``delta = +1`` for E4 (a paper E4 byte read as a
  native E4 byte is exactly twice the value) and ``delta = 0`` for E5.
* ``CONV_NATIVE``: Eq. 3 with the native format's own ``max_num`` (448 /
  57344) and ``delta = 0``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

P_E4, P_E5, N_E4, N_E5 = 0, 1, 2, 3
E4, E5 = 0, 1
CONV_PAPER, CONV_NATIVE = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fp8_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile ``fp8_oracle.c`` with gcc (-O2 -fopenmp) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        c = ctypes
        _lib.orc_decode.restype = c.c_double
        _lib.orc_decode.argtypes = [c.c_int, c.c_uint]
        _lib.orc_max_num.restype = c.c_double
        _lib.orc_max_num.argtypes = [c.c_int]
        _lib.orc_encode.restype = c.c_uint
        _lib.orc_encode.argtypes = [c.c_int, c.c_double]
        _lib.orc_f32_to_bf16.restype = c.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [c.c_float]
        _lib.orc_amax.restype = c.c_float
        _lib.orc_amax.argtypes = [c.c_void_p, c.c_int, c.c_int64, c.c_int64, c.c_int64]
        _lib.orc_scaling_bias.restype = c.c_int
        _lib.orc_scaling_bias.argtypes = [c.c_float, c.c_double, c.c_int]
        _lib.orc_cast.restype = None
        _lib.orc_cast.argtypes = [c.c_void_p, c.c_int, c.c_int64, c.c_int64, c.c_int64, c.c_int, c.c_int,
                                  c.c_void_p, c.c_void_p]
        gemm_args = [c.c_void_p, c.c_int, c.c_int, c.c_void_p, c.c_int, c.c_int]
        tail = [c.c_int64, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib.orc_linear_fwd.restype = None
        _lib.orc_linear_fwd.argtypes = gemm_args + [c.c_void_p] + tail
        _lib.orc_linear_dgrad.restype = None
        _lib.orc_linear_dgrad.argtypes = gemm_args + tail
        _lib.orc_linear_wgrad.restype = None
        _lib.orc_linear_wgrad.argtypes = gemm_args + tail
        _lib.orc_linear_samples.restype = None
        _lib.orc_linear_samples.argtypes = [c.c_int] + gemm_args + [c.c_void_p, c.c_int64, c.c_int64, c.c_int64,
                                                                    c.c_void_p, c.c_void_p, c.c_int64,
                                                                    c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib.orc_num_threads.restype = c.c_int
    return _lib


def num_threads() -> int:
    return int(_L().orc_num_threads())


# ----------------------------------------------------------------------------
# formats
# ----------------------------------------------------------------------------

def decode(fmt: int, code: int) -> float:
    return float(_L().orc_decode(fmt, int(code) & 0xFF))


def decode_table(fmt: int) -> np.ndarray:
    return np.array([decode(fmt, c) for c in range(256)], dtype=np.float64)


def encode(fmt: int, value: float) -> int:
    return int(_L().orc_encode(fmt, float(value)))


def max_num(fmt: int) -> float:
    return float(_L().orc_max_num(fmt))


def native_format(kind: int) -> int:
    return N_E4 if kind == E4 else N_E5


def paper_format(kind: int) -> int:
    return P_E4 if kind == E4 else P_E5


def bias_max_num(kind: int, conv: int) -> float:
    """``max_num`` that Eq. 3 uses under a convention."""
    return max_num(paper_format(kind) if conv == CONV_PAPER else native_format(kind))


def delta(kind: int, conv: int) -> int:
    """Format shift between the paper-convention bias and the shift applied to
    produce native bytes."""
    return 1 if (conv == CONV_PAPER and kind == E4) else 0


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    f = _L().orc_f32_to_bf16
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def f32_to_bf16_bits_np(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (NaN stays NaN), on whole arrays; the same rule as
    ``orc_f32_to_bf16`` (tests/test_oracle_gemm.py holds the two together)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return np.where(nan, (u >> 16) | 0x40, rounded).astype(np.uint16)


# ----------------------------------------------------------------------------
# amax, bias, cast
# ----------------------------------------------------------------------------

def _tensor(x: np.ndarray):
    """A 2-D input tensor and its type id: bf16 is passed as uint16 bit
    patterns, fp16 as numpy float16, fp32 as numpy float32."""
    assert x.ndim == 2
    dt = {np.dtype(np.uint16): 0, np.dtype(np.float16): 1, np.dtype(np.float32): 2}[x.dtype]
    return np.ascontiguousarray(x), dt


def amax(x_bits: np.ndarray) -> float:
    x, dt = _tensor(x_bits)
    return float(_L().orc_amax(x.ctypes.data, dt, x.shape[0], x.shape[1], x.shape[1]))


def scaling_bias(amax_value: float, kind: int, conv: int = CONV_PAPER, margin: int = 0) -> int:
    return int(_L().orc_scaling_bias(float(np.float32(amax_value)), bias_max_num(kind, conv), int(margin)))


def history_bias(amax_window, kind: int, conv: int = CONV_PAPER, margin: int = 0) -> int:
    """Amax-history scaling (Section 3: scale from earlier steps' amax instead of a second pass over the
    tensor): the bias for the next step is Eq. 3 on the largest amax of the window, minus the margin."""
    return scaling_bias(max(float(a) for a in amax_window), kind, conv, margin)


def bias_mode(biases):
    """The statistic Appendix G plots per tensor: the mode of its scaling bias over the samples.  Returns
    (mode, how often it occurs); the smaller bias on a tie, (0, 0) for no samples."""
    counts = {}
    for b in biases:
        counts[int(b)] = counts.get(int(b), 0) + 1
    if not counts:
        return 0, 0
    top = max(counts.values())
    return min(b for b, c in counts.items() if c == top), top


def cast(x_bits: np.ndarray, shift: int, fmt: int, transposed: bool = False):
    """codes = encode_fmt(x * 2^shift); returns y[rows, cols] and, if asked,
    also y_t[cols, rows]."""
    x, dt = _tensor(x_bits)
    rows, cols = x.shape
    y = np.empty((rows, cols), dtype=np.uint8)
    y_t = np.empty((cols, rows), dtype=np.uint8) if transposed else None
    _L().orc_cast(x.ctypes.data, dt, rows, cols, cols, int(shift), fmt, y.ctypes.data,
                  y_t.ctypes.data if transposed else None)
    return (y, y_t) if transposed else y


def quantise(x_bits: np.ndarray, kind: int, conv: int = CONV_PAPER, margin: int = 0, transposed: bool = False):
    """amax -> bias -> scale -> cast of one tensor (Section 2.3 then 2.1).
    Returns (amax, bias, native bytes[, transposed native bytes])."""
    a = amax(x_bits)
    b = scaling_bias(a, kind, conv, margin)
    out = cast(x_bits, b + delta(kind, conv), native_format(kind), transposed)
    return (a, b) + (out if transposed else (out,))


# ----------------------------------------------------------------------------
# matmuls
# ----------------------------------------------------------------------------

class GemmResult:
    def __init__(self, shape):
        self.f64 = np.empty(shape, dtype=np.float64)
        self.f32 = np.empty(shape, dtype=np.float32)
        self.bf16 = np.empty(shape, dtype=np.uint16)
        self.abs_sum = np.empty(shape, dtype=np.float64)

    def _ptrs(self):
        return (self.f64.ctypes.data, self.f32.ctypes.data, self.bf16.ctypes.data, self.abs_sum.ctypes.data)


def _u8(a):
    assert a.dtype == np.uint8 and a.ndim == 2
    return np.ascontiguousarray(a)


def linear_fwd(x8, s_x, w8, s_w, bias_vec=None, fx=N_E4, fw=N_E4) -> GemmResult:
    x8, w8 = _u8(x8), _u8(w8)
    T, K = x8.shape
    N, K2 = w8.shape
    assert K == K2
    res = GemmResult((T, N))
    bv = None
    if bias_vec is not None:
        bv = np.ascontiguousarray(bias_vec, dtype=np.float64)
        assert bv.shape == (N,)
    _L().orc_linear_fwd(x8.ctypes.data, fx, int(s_x), w8.ctypes.data, fw, int(s_w),
                        bv.ctypes.data if bv is not None else None, T, K, N, *res._ptrs())
    return res


def linear_dgrad(dy8, s_g, w8, s_w, fg=N_E5, fw=N_E4) -> GemmResult:
    dy8, w8 = _u8(dy8), _u8(w8)
    T, N = dy8.shape
    N2, K = w8.shape
    assert N == N2
    res = GemmResult((T, K))
    _L().orc_linear_dgrad(dy8.ctypes.data, fg, int(s_g), w8.ctypes.data, fw, int(s_w), T, K, N, *res._ptrs())
    return res


def linear_wgrad(dy8, s_g, x8, s_x, fg=N_E5, fx=N_E4) -> GemmResult:
    dy8, x8 = _u8(dy8), _u8(x8)
    T, N = dy8.shape
    T2, K = x8.shape
    assert T == T2
    res = GemmResult((N, K))
    _L().orc_linear_wgrad(dy8.ctypes.data, fg, int(s_g), x8.ctypes.data, fx, int(s_x), T, K, N, *res._ptrs())
    return res


FWD, DGRAD, WGRAD = 0, 1, 2


def linear_samples(kind, a8, fa, s_a, b8, fb, s_b, rows, cols, bias_vec=None) -> GemmResult:
    """The matmul definitions evaluated at listed (row, col) output positions.
    kind FWD: a8 = X8[T,K], b8 = W8[N,K]; DGRAD: a8 = dY8[T,N], b8 = W8[N,K];
    WGRAD: a8 = dY8[T,N], b8 = X8[T,K]."""
    a8, b8 = _u8(a8), _u8(b8)
    if kind == FWD:
        (T, K), (N, _) = a8.shape, b8.shape
    elif kind == DGRAD:
        (T, N), (_, K) = a8.shape, b8.shape
    else:
        (T, N), (_, K) = a8.shape, b8.shape
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    assert rows.shape == cols.shape and rows.ndim == 1
    res = GemmResult(rows.shape)
    bv = None
    if bias_vec is not None:
        bv = np.ascontiguousarray(bias_vec, dtype=np.float64)
    _L().orc_linear_samples(kind, a8.ctypes.data, fa, int(s_a), b8.ctypes.data, fb, int(s_b),
                            bv.ctypes.data if bv is not None else None, T, K, N,
                            rows.ctypes.data, cols.ctypes.data, rows.size, *res._ptrs())
    return res


# ----------------------------------------------------------------------------
# the same matmul definitions with numpy's float64 matmul as the summation step
# ----------------------------------------------------------------------------
# Every product of two FP8 values is a small multiple of a power of two, so a float64 sum of them is exact as long
# as the terms' exponents span less than float64's 53 bits; with E5 x E4 operands over the formats' full range
# they can span more, and a BLAS may then differ from the plain C loops by a rounding of the float64 sum (a
# relative 2^-53 or so of sum |a*b|: nine orders of magnitude inside the 2^-14 bar).  So these functions return
# what the plain C loops return exactly after the rounding to float32 / bf16 except at a float64-level tie, and to
# 2^-50 relative in float64 (tests/test_oracle_gemm.py checks both); they exist because the C loops need minutes
# where a 24-layer trajectory or a full-size layer has to be checked.

class _NpResult:
    def __init__(self, f64, abs_sum):
        self.f64 = f64
        self.abs_sum = abs_sum
        self.f32 = f64.astype(np.float32)
        self.bf16 = f32_to_bf16_bits_np(self.f32)


def _matmul_unscale(A, B_t, shift_sum, bias_vec=None):
    f64 = np.ldexp(A @ B_t, -shift_sum)
    abs_sum = np.ldexp(np.abs(A) @ np.abs(B_t), -shift_sum)
    if bias_vec is not None:
        bv = np.asarray(bias_vec, dtype=np.float64)
        f64 = f64 + bv[None, :]
        abs_sum = abs_sum + np.abs(bv)[None, :]
    return _NpResult(f64, abs_sum)


def linear_fwd_np(x8, s_x, w8, s_w, bias_vec=None, fx=N_E4, fw=N_E4):
    """Y = (X8 . W8^T) * 2^-(s_x+s_w) (+ bias_vec)."""
    return _matmul_unscale(decode_table(fx)[_u8(x8)], decode_table(fw)[_u8(w8)].T, int(s_x) + int(s_w), bias_vec)


def linear_dgrad_np(dy8, s_g, w8, s_w, fg=N_E5, fw=N_E4):
    """dX = (dY8 . W8) * 2^-(s_g+s_w)."""
    return _matmul_unscale(decode_table(fg)[_u8(dy8)], decode_table(fw)[_u8(w8)], int(s_g) + int(s_w))


def linear_wgrad_np(dy8, s_g, x8, s_x, fg=N_E5, fx=N_E4):
    """dW = (dY8^T . X8) * 2^-(s_g+s_x)."""
    return _matmul_unscale(decode_table(fg)[_u8(dy8)].T, decode_table(fx)[_u8(x8)], int(s_g) + int(s_x))


# ----------------------------------------------------------------------------
# FP16 accumulation (Fig. 3b and Section 2.4)
# ----------------------------------------------------------------------------
# The paper's own matmul takes FP8 inputs, accumulates the partial results in FP16 and outputs FP16 (Fig. 3b);
# Section 2.4 explains that this is where loss scaling comes back in, and Section 3.2 that the two backward matmuls
# can overflow FP16 unless a margin lowers the bias of the E5 operand.  The paper does not say how many products
# the hardware adds before it rounds to FP16.  Reading taken here, with the granularity an explicit argument:
# the products of `chunk` consecutive contraction indices are summed exactly; every such partial sum is added to
# a running FP16 accumulator with one rounding to FP16 (nearest even; beyond 65504 the accumulator becomes
# infinite and stays so); the FP16 accumulator is then unscaled by 2^-(s_a + s_b) in FP16 (Eq. 2 on the FP16
# output: exact unless the result leaves FP16's normal range, where it rounds once or becomes infinite / zero).
# chunk = 1 is a purely sequential FP16 accumulation.

class Fp16AccResult:
    def __init__(self, f16, peak, shift_sum):
        self.f16 = f16                          # numpy float16: what an FP16 output tensor would hold
        self.f64 = f16.astype(np.float64)
        self.overflowed = ~np.isfinite(self.f64)
        # largest magnitude the running FP16 sum went through, in the output's (unscaled) units: one FP16 step at
        # THAT magnitude is the resolution of the whole accumulation, however small the final value is
        self.peak = np.ldexp(peak, -int(shift_sum))


def _matmul_fp16acc(A, B_t, shift_sum, chunk):
    """A [M, Kc] and B_t [Kc, N] decoded to float64; Kc is the contraction."""
    assert chunk >= 1
    M, Kc = A.shape
    acc = np.zeros((M, B_t.shape[1]), dtype=np.float16)
    peak = np.zeros(acc.shape, dtype=np.float64)
    for k0 in range(0, Kc, chunk):
        partial = A[:, k0:k0 + chunk] @ B_t[k0:k0 + chunk, :]          # exact: few terms, each a short dyadic number
        with np.errstate(over="ignore", invalid="ignore"):
            acc = (acc.astype(np.float64) + partial).astype(np.float16)    # one rounding to FP16 per chunk
        peak = np.maximum(peak, np.abs(acc.astype(np.float64)))
    with np.errstate(over="ignore", under="ignore"):
        out = np.ldexp(acc.astype(np.float64), -int(shift_sum)).astype(np.float16)
    return Fp16AccResult(out, peak, shift_sum)


def linear_fwd_fp16acc(x8, s_x, w8, s_w, chunk=128, fx=N_E4, fw=N_E4):
    """Y = FP16-accumulated (X8 . W8^T), unscaled in FP16."""
    return _matmul_fp16acc(decode_table(fx)[_u8(x8)], decode_table(fw)[_u8(w8)].T, int(s_x) + int(s_w), chunk)


def linear_dgrad_fp16acc(dy8, s_g, w8, s_w, chunk=128, fg=N_E5, fw=N_E4):
    """dX = FP16-accumulated (dY8 . W8), unscaled in FP16."""
    return _matmul_fp16acc(decode_table(fg)[_u8(dy8)], decode_table(fw)[_u8(w8)], int(s_g) + int(s_w), chunk)


def linear_wgrad_fp16acc(dy8, s_g, x8, s_x, chunk=128, fg=N_E5, fx=N_E4):
    """dW = FP16-accumulated (dY8^T . X8), unscaled in FP16."""
    return _matmul_fp16acc(decode_table(fg)[_u8(dy8)].T, decode_table(fx)[_u8(x8)], int(s_g) + int(s_x), chunk)
