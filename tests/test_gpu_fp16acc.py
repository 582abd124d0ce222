"""GPU parity: fp8_linear_f16acc (the paper's FP16-accumulation regime, emulated) against the oracle's
linear_*_fp16acc on the same FP8 bytes and biases.

The partial sum of one slice comes from the tensor cores in FP32 (exact to about 2^-22 of its absolute sum) where the
oracle's is exact, and the FP16 rounding of "running sum + partial sum" goes through one FP32 addition first; either can
flip a rounding that sits within a hair of a tie.  Bar: at least 99 % of the outputs bit-identical; none further from
the oracle than two FP16 steps AT THE LARGEST MAGNITUDE ITS RUNNING SUM WENT THROUGH (a flipped rounding of a large
intermediate sum is many steps of a final value that cancelled down to something small); and the same outputs infinite
(an output may differ in that only if the oracle's finite value is within one step of FP16's maximum)."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import bits_of, u8
from paper_2309_17224_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2309_17224_b200 import fp8lin
    return fp8lin


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0)
    yield c
    c.close()


def _f16_ordinal(x: np.ndarray) -> np.ndarray:
    b = x.view(np.uint16).astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def _compare(got: torch.Tensor, ref: "O.Fp16AccResult", what):
    g = got.cpu().numpy()
    if g.dtype == np.float32:
        assert np.array_equal(g.astype(np.float16).astype(np.float32), g, equal_nan=True), "FP32 output must hold FP16 values"
        g = g.astype(np.float16)
    r = ref.f16
    inf_g, inf_r = np.isinf(g), np.isinf(r)
    differ = inf_g != inf_r
    if differ.any():   # only at the very edge of FP16's range
        edge = np.abs(np.where(inf_r, g, r).astype(np.float64)) >= 65472.0
        assert edge[differ].all(), what
    fin = ~(inf_g | inf_r)
    d = np.abs(_f16_ordinal(g[fin]) - _f16_ordinal(r[fin]))
    peak = np.maximum(ref.peak[fin], np.abs(ref.f64[fin]))
    step = np.exp2(np.floor(np.log2(np.maximum(peak, 2.0 ** -14))) - 10)      # one FP16 step at that magnitude
    err = np.abs(g[fin].astype(np.float64) - ref.f64[fin])
    assert d.size == 0 or bool((err <= 2 * step).all()), (what, float((err / step).max()))
    same = float((d == 0).mean()) if d.size else 1.0
    assert same >= 0.99, (what, same)
    return same, float(inf_r.mean())


class Fixed:
    """A tensor cast under a given bias (FP8-CSCALE) on the GPU, with the oracle's bytes checked."""

    def __init__(self, ctx, lib, x, kind, bias):
        self.bias = torch.tensor([bias], dtype=torch.int32, device="cuda")
        self.y = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        (ctx.cast_e4 if kind == O.E4 else ctx.cast_e5)(x, self.bias, y=self.y)
        self.shift = bias + O.delta(kind, O.CONV_PAPER)
        self.ref = O.cast(bits_of(x), self.shift, O.native_format(kind))
        assert np.array_equal(u8(self.y), self.ref)


def _amax_bias(x, kind, margin=0):
    return O.scaling_bias(O.amax(bits_of(x)), kind, O.CONV_PAPER, margin)


@pytest.mark.parametrize("T,K,N", [(200, 512, 304), (64, 1040, 512), (300, 2304, 272), (130, 128, 272)])
@pytest.mark.parametrize("chunk", [128, 256, 1024])
def test_three_matmuls_with_fp16_accumulation_match_the_oracle(ctx, lib, T, K, N, chunk):
    x = I.normal_bf16(T, K, 1.0, 5, 1, "cuda", outlier_frac=0.01, outlier_scale=20.0)
    w = I.normal_bf16(N, K, 0.02, 5, 2, "cuda")
    g = I.normal_bf16(T, N, 1e-3, 5, 3, "cuda")
    # biases that keep the scaled accumulators inside FP16 (weights and activations well below their maximum, the
    # gradient at FP8-AMAX minus a margin of 3)
    qx = Fixed(ctx, lib, x, O.E4, _amax_bias(x, O.E4) - 5)
    qw = Fixed(ctx, lib, w, O.E4, _amax_bias(w, O.E4) - 5)
    qg = Fixed(ctx, lib, g, O.E5, _amax_bias(g, O.E5, margin=3) - 4)
    cases = ((lib.MM_FWD, qx, qw, (T, N), O.linear_fwd_fp16acc(qx.ref, qx.shift, qw.ref, qw.shift, chunk=chunk)),
             (lib.MM_DGRAD, qg, qw, (T, K), O.linear_dgrad_fp16acc(qg.ref, qg.shift, qw.ref, qw.shift, chunk=chunk)),
             (lib.MM_WGRAD, qg, qx, (N, K), O.linear_wgrad_fp16acc(qg.ref, qg.shift, qx.ref, qx.shift, chunk=chunk)))
    for kind, a, b, shape, ref in cases:
        for dt in (torch.float16, torch.float32):
            out = torch.full(shape, float("nan"), dtype=dt, device="cuda")
            ctx.linear_f16acc(kind, a.y, a.bias, b.y, b.bias, out, T, K, N, chunk=chunk)
            same, infs = _compare(out, ref, (kind, dt))
            assert infs == 0.0                         # this regime must stay finite on both sides
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_margin_decides_whether_the_input_gradient_overflows_fp16(ctx, lib):
    """Section 3.2 on the GPU: the gradient at plain FP8-AMAX sits next to FP16's maximum and the FP16 accumulator of
    dX = dY8 . W8 overflows; a margin of 3 leaves room.  (Weights under a constant bias, so that the gradient alone
    decides.)  Same infinities as the oracle in both runs."""
    T, K, N = 192, 256, 512
    g = I.normal_bf16(T, N, 1e-4, 11, 3, "cuda")
    w = I.normal_bf16(N, K, 0.2, 11, 2, "cuda")
    qw = Fixed(ctx, lib, w, O.E4, 0)
    seen = {}
    for margin in (0, 3):
        qg = Fixed(ctx, lib, g, O.E5, _amax_bias(g, O.E5, margin=margin))
        ref = O.linear_dgrad_fp16acc(qg.ref, qg.shift, qw.ref, qw.shift, chunk=128)
        out = torch.empty((T, K), dtype=torch.float16, device="cuda")
        ctx.linear_f16acc(lib.MM_DGRAD, qg.y, qg.bias, qw.y, qw.bias, out, T, K, N, chunk=128)
        _compare(out, ref, margin)
        seen[margin] = float(torch.isinf(out).float().mean().item())
    assert seen[0] > 0.05 and seen[3] == 0.0, seen


def test_fp16_accumulation_differs_from_fp32_accumulation_as_the_oracle_says(ctx, lib):
    """The emulation must not be the FP32 path in disguise: on a long contraction the FP16 running sum loses bits that
    the FP32 accumulator keeps, by the amount the oracle predicts."""
    T, K, N = 128, 8192, 256
    x = I.normal_bf16(T, K, 1.0, 21, 1, "cuda")
    w = I.normal_bf16(N, K, 0.02, 21, 2, "cuda")
    qx = Fixed(ctx, lib, x, O.E4, _amax_bias(x, O.E4) - 6)
    qw = Fixed(ctx, lib, w, O.E4, _amax_bias(w, O.E4) - 6)
    ref16 = O.linear_fwd_fp16acc(qx.ref, qx.shift, qw.ref, qw.shift, chunk=128)
    exact = O.linear_fwd_np(qx.ref, qx.shift, qw.ref, qw.shift).f64
    out = torch.empty((T, N), dtype=torch.float16, device="cuda")
    ctx.linear_f16acc(lib.MM_FWD, qx.y, qx.bias, qw.y, qw.bias, out, T, K, N, chunk=128)
    _compare(out, ref16, "long contraction")
    err_gpu = np.abs(out.cpu().numpy().astype(np.float64) - exact)
    half_ulp = np.abs(exact) * 2.0 ** -11
    assert (err_gpu > 2 * half_ulp).mean() > 0.2     # far more than one output rounding: 64 roundings of a running sum


def test_f16acc_argument_errors(ctx, lib):
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    a8 = torch.zeros((64, 128), dtype=torch.uint8, device="cuda")
    b8 = torch.zeros((48, 128), dtype=torch.uint8, device="cuda")
    out = torch.zeros((64, 48), dtype=torch.float16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_f16acc(lib.MM_FWD, a8, b, b8, b, out, 64, 128, 48, chunk=100)      # not a multiple of 128
    assert e.value.status == lib.ERR_SHAPE
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_f16acc(lib.MM_FWD, a8, b, b8, b, out.to(torch.bfloat16), 64, 128, 48)   # bf16 cannot hold FP16 values
    assert e.value.status == lib.ERR_UNSUPPORTED
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_f16acc(7, a8, b, b8, b, out, 64, 128, 48)
    assert e.value.status == lib.ERR_DTYPE
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_f16acc(lib.MM_FWD, a8, None, b8, b, out, 64, 128, 48)
    assert e.value.status == lib.ERR_NULL
    ctx.linear_f16acc(lib.MM_FWD, a8, b, b8, b, out, 64, 128, 48)
    assert bool((out == 0).all()) and ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
