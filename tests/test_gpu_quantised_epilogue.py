"""GPU parity: matmuls whose epilogue writes the consumer's FP8 bytes for a bias
known before the launch (amax-history scaling, Section 3).

The 16-bit tensor the bytes are made from must meet the usual matmul bars
against the oracle; the bytes must equal, bit for bit, the oracle's cast of
that stored 16-bit tensor under the given bias; the amax must be the amax of
what was stored; the saturation flag must be raised exactly when the oracle's
scaled values leave the format's range.
"""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import stack as OS
from helpers import assert_bf16_within_one_ulp, assert_codes_equal, bf16_ordinal, bits_of, u8
from paper_2309_17224_b200 import inputs as I
from test_gpu_linear import Quantised, _layer

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


def _dev_i32(v):
    return torch.tensor([v], dtype=torch.int32, device="cuda")


def _check_bytes(ctx, lib, z, z8, amax_z, bias, kind, conv, expect_clip):
    """expect_clip: True / False where the choice of bias settles it, None where it depends on the mantissa of
    the amax (then the documented rule decides: a scaled value that rounds beyond the largest finite code)."""
    zb = bits_of(z)
    fmt = O.native_format(kind)
    shift = bias + O.delta(kind, conv)
    want = O.cast(zb, shift, fmt)
    assert_codes_equal(u8(z8), want, fmt)
    assert float(amax_z.item()) == O.amax(zb)
    scaled = np.abs(OS.bf16_to_f64(zb)) * 2.0 ** shift
    clip = bool((scaled > 464.0).any()) if kind == O.E4 else bool((scaled >= 61440.0).any())
    if expect_clip is not None:
        assert clip == expect_clip
    flags = ctx.device_flags(clear=True)
    assert flags & lib.FLAG_TIMEOUT == 0
    assert bool(flags & lib.FLAG_SATURATED) == clip


SHAPES = [(256, 768, 768), (144, 272, 528), (400, 1040, 784), (64, 1024, 512), (16, 2048, 48), (300, 128, 1296)]


@pytest.mark.parametrize("T,K,N", SHAPES)
@pytest.mark.parametrize("act", ["none", "gelu"])
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_forward_with_quantised_output(ctx, lib, T, K, N, act, conv):
    qx, qw, _ = _layer(ctx, T, K, N, conv, seed=4100 + T)
    bv = I.normal_bf16(1, N, 0.1, 9, 7, "cuda").reshape(N)
    ref = O.linear_fwd_np(qx.ref, qx.shift, qw.ref, qw.shift, bias_vec=bv.double().cpu().numpy())
    gelu = act == "gelu"
    # the bias a perfect prediction gives (from the oracle's own z), one that clips, one with headroom
    z_ref = OS.gelu_bits(ref.bf16) if gelu else ref.bf16
    exact = O.scaling_bias(O.amax(z_ref), O.E4, conv)
    kept = None
    for bias, clip in ((exact, None), (exact + 2, True), (exact - 3, False)):
        y_pre = torch.full((T, N), float("nan"), dtype=torch.bfloat16, device="cuda") if gelu else None
        z = torch.full((T, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        z8 = torch.full((T, N), 0xAA, dtype=torch.uint8, device="cuda")
        amax_z = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        ctx.linear_fwd_q(qx.y, qx.bias, qw.y, qw.bias, z8, _dev_i32(bias), y_pre=y_pre, z=z, bias_vec=bv,
                         d_amax_z=amax_z, act=lib.ACT_GELU if gelu else lib.ACT_NONE, conv=conv)
        if gelu:
            assert_bf16_within_one_ulp(bits_of(y_pre), ref)
            d = np.abs(bf16_ordinal(bits_of(z)) - bf16_ordinal(OS.gelu_bits(bits_of(y_pre))))
            assert d.max() <= 1, d.max()
        else:
            assert_bf16_within_one_ulp(bits_of(z), ref)
        if kept is None:
            kept = bits_of(z)
        else:
            assert np.array_equal(bits_of(z), kept)      # the 16-bit tensor does not depend on the bias
        _check_bytes(ctx, lib, z, z8, amax_z, bias, O.E4, conv, clip)
    # the same bytes without asking for any 16-bit tensor
    z8_only = torch.full((T, N), 0x55, dtype=torch.uint8, device="cuda")
    ctx.linear_fwd_q(qx.y, qx.bias, qw.y, qw.bias, z8_only, _dev_i32(exact - 3), bias_vec=bv,
                     act=lib.ACT_GELU if gelu else lib.ACT_NONE, conv=conv)
    assert torch.equal(z8_only, z8)
    assert ctx.device_flags(clear=True) == 0


@pytest.mark.parametrize("T,K,N", [(256, 768, 768), (144, 272, 528), (400, 1040, 784), (16, 48, 2048)])
@pytest.mark.parametrize("act", ["none", "gelu"])
@pytest.mark.parametrize("layout", ["t", "mn"])
def test_input_gradient_with_quantised_output(ctx, lib, T, K, N, act, layout):
    conv = O.CONV_PAPER
    qx, qw, qg = _layer(ctx, T, K, N, conv, seed=5100 + T)
    ref = O.linear_dgrad_np(qg.ref, qg.shift, qw.ref, qw.shift)
    gelu = act == "gelu"
    y_pre = I.normal_bf16(T, K, 1.5, 13, 9, "cuda") if gelu else None
    if gelu:
        z_ref = OS.f64_to_bf16(OS.bf16_to_f64(ref.bf16) * OS.gelu_grad(bits_of(y_pre)))
    else:
        z_ref = ref.bf16
    exact = O.scaling_bias(O.amax(z_ref), O.E5, conv)
    w8, w8t = (None, qw.y_t) if layout == "t" else (qw.y, None)
    for bias, clip in ((exact, None), (exact + 2, True), (exact - 4, False)):
        dx = torch.full((T, K), float("nan"), dtype=torch.bfloat16, device="cuda") if gelu else None
        g = torch.full((T, K), float("nan"), dtype=torch.bfloat16, device="cuda")
        g8 = torch.full((T, K), 0xAA, dtype=torch.uint8, device="cuda")
        amax_g = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        ctx.linear_dgrad_q(qg.y, qg.bias, w8, w8t, qw.bias, g8, _dev_i32(bias), y_pre=y_pre, dx=dx, g=g,
                           d_amax_g=amax_g, act=lib.ACT_GELU if gelu else lib.ACT_NONE, conv=conv)
        if gelu:
            assert_bf16_within_one_ulp(bits_of(dx), ref)
            want = OS.f64_to_bf16(OS.bf16_to_f64(bits_of(dx)) * OS.gelu_grad(bits_of(y_pre)))
            d = np.abs(bf16_ordinal(bits_of(g)) - bf16_ordinal(want))
            assert d.max() <= 1, d.max()
        else:
            assert_bf16_within_one_ulp(bits_of(g), ref)
        _check_bytes(ctx, lib, g, g8, amax_g, bias, O.E5, conv, clip)


def test_quantised_output_feeds_the_next_matmul(ctx, lib):
    """Two chained layers: the second consumes the bytes the first one's epilogue wrote, and gives exactly what
    it gives on bytes cast from the stored 16-bit activation in a separate pass."""
    T, d = 384, 512
    qx, qw1, _ = _layer(ctx, T, d, d, O.CONV_PAPER, seed=77)
    w2 = I.normal_bf16(d, d, 0.02, 78, 2, "cuda")
    qw2 = Quantised(ctx, w2, O.E4, O.CONV_PAPER)
    z = torch.empty((T, d), dtype=torch.bfloat16, device="cuda")
    z8 = torch.empty((T, d), dtype=torch.uint8, device="cuda")
    amax_z = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias_z = _dev_i32(3)
    ctx.linear_fwd_q(qx.y, qx.bias, qw1.y, qw1.bias, z8, bias_z, z=z, d_amax_z=amax_z, act=lib.ACT_GELU)
    z8_sep = torch.empty_like(z8)
    ctx.cast_e4(z, bias_z, y=z8_sep)
    assert torch.equal(z8, z8_sep)
    y_a = torch.empty((T, d), dtype=torch.float32, device="cuda")
    y_b = torch.empty_like(y_a)
    ctx.linear_fwd(z8, bias_z, qw2.y, qw2.bias, y_a)
    ctx.linear_fwd(z8_sep, bias_z, qw2.y, qw2.bias, y_b)
    assert torch.equal(y_a, y_b)
    # the history update: the bias Eq. 3 gives for the amax that came out of the first launch
    b_next = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.scaling_bias(amax_z, lib.E4, lib.CONV_PAPER, 0, b_next)
    assert int(b_next.item()) == O.scaling_bias(O.amax(bits_of(z)), O.E4)
    assert ctx.device_flags(clear=True) & ~lib.FLAG_SATURATED == 0


def test_quantised_output_argument_errors(ctx, lib):
    x8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    w8 = torch.zeros((48, 64), dtype=torch.uint8, device="cuda")
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    z8 = torch.zeros((32, 48), dtype=torch.uint8, device="cuda")
    y = torch.zeros((32, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8, b, None, b)                             # the bytes are mandatory
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8, b, z8, None)                            # so is the bias
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8, b, z8, b, y_pre=y)                      # no activation: no separate pre-activation
    assert e.value.status == lib.ERR_UNSUPPORTED
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8, b, z8, b, act=5)
    assert e.value.status == lib.ERR_DTYPE
    w8_odd = torch.zeros((40, 64), dtype=torch.uint8, device="cuda")        # N = 40: rows of bytes not 16-byte multiples
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8_odd, b, torch.zeros((32, 40), dtype=torch.uint8, device="cuda"), b)
    assert e.value.status == lib.ERR_ALIGN
    g8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    dy8 = torch.zeros((32, 48), dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad_q(dy8, b, w8, None, b, g8, b, act=lib.ACT_GELU)    # GELU' needs the pre-activation
    assert e.value.status == lib.ERR_NULL
    ctx.linear_fwd_q(x8, b, w8, b, z8, b, z=y)
    assert bool((y == 0).all()) and bool((z8 == 0).all()) and ctx.device_flags(clear=True) == 0
