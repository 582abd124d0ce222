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


def _interleaved_weight(ctx, F, K, conv, seed):
    """A gate/up weight pair merged into the 32-row block layout, quantised on the GPU and by the oracle."""
    gate = I.normal_bf16(F, K, 0.02, seed, 2, "cuda")
    up = I.normal_bf16(F, K, 0.02, seed, 4, "cuda")
    return Quantised(ctx, I.interleave32(gate, up).contiguous(), O.E4, conv)


@pytest.mark.parametrize("T,K,F", [(256, 768, 384), (144, 272, 96), (400, 1040, 416), (64, 1024, 256), (300, 128, 32)])
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_forward_with_swiglu_epilogue(ctx, lib, T, K, F, conv):
    """z = SiLU(gate) * up out of the forward epilogue (weight rows in blocks of 32 gate, 32 up): the
    pre-activation meets the forward bar, z is within one bf16 ulp of float64 SwiGLU of the GPU's own
    pre-activation bits, bytes / amax / saturation as for every quantised output."""
    N = 2 * F
    x = I.normal_bf16(T, K, 1.0, 6100 + T, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0)
    qx = Quantised(ctx, x, O.E4, conv)
    qw = _interleaved_weight(ctx, F, K, conv, 6100 + T)
    ref = O.linear_fwd_np(qx.ref, qx.shift, qw.ref, qw.shift)
    exact = O.scaling_bias(O.amax(OS.swiglu_bits(ref.bf16)), O.E4, conv)
    kept = None
    for bias, clip in ((exact, None), (exact + 2, True), (exact - 3, False)):
        y_pre = torch.full((T, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        z = torch.full((T, F), float("nan"), dtype=torch.bfloat16, device="cuda")
        z8 = torch.full((T, F), 0xAA, dtype=torch.uint8, device="cuda")
        amax_z = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        ctx.linear_fwd_q(qx.y, qx.bias, qw.y, qw.bias, z8, _dev_i32(bias), y_pre=y_pre, z=z, d_amax_z=amax_z,
                         act=lib.ACT_SWIGLU, conv=conv)
        assert_bf16_within_one_ulp(bits_of(y_pre), ref)
        d = np.abs(bf16_ordinal(bits_of(z)) - bf16_ordinal(OS.swiglu_bits(bits_of(y_pre))))
        assert d.max() <= 1, d.max()
        if kept is None:
            kept = bits_of(z)
        else:
            assert np.array_equal(bits_of(z), kept)
        _check_bytes(ctx, lib, z, z8, amax_z, bias, O.E4, conv, clip)
    # the unquantised twin gives the same z and amax; bytes alone give the same bytes
    z2 = torch.full((T, F), float("nan"), dtype=torch.bfloat16, device="cuda")
    amax2 = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.linear_fwd_act(qx.y, qx.bias, qw.y, qw.bias, None, z2, d_amax_act=amax2, act=lib.ACT_SWIGLU, conv=conv)
    assert np.array_equal(bits_of(z2), kept) and float(amax2.item()) == float(amax_z.item())
    z8_only = torch.full((T, F), 0x55, dtype=torch.uint8, device="cuda")
    ctx.linear_fwd_q(qx.y, qx.bias, qw.y, qw.bias, z8_only, _dev_i32(exact - 3), act=lib.ACT_SWIGLU, conv=conv)
    assert torch.equal(z8_only, z8)
    assert ctx.device_flags(clear=True) == 0


@pytest.mark.parametrize("T,F,N", [(256, 384, 768), (144, 96, 272), (400, 416, 1040), (16, 2048, 48), (300, 32, 128)])
@pytest.mark.parametrize("layout", ["t", "mn"])
def test_input_gradient_with_swiglu_backward_epilogue(ctx, lib, T, F, N, layout):
    """dz[T, F] = dY8 . W8 (the down projection's input gradient); the epilogue turns it into the gradients of the
    stored gate / up pre-activations [T, 2F] (block layout), their E5 bytes and amax."""
    conv = O.CONV_PAPER
    g = I.normal_bf16(T, N, 1e-3, 7100 + T, 3, "cuda")
    w = I.normal_bf16(N, F, 0.02, 7100 + T, 2, "cuda")
    qg, qw = Quantised(ctx, g, O.E5, conv), Quantised(ctx, w, O.E4, conv)
    ref = O.linear_dgrad_np(qg.ref, qg.shift, qw.ref, qw.shift)
    y_pre = I.normal_bf16(T, 2 * F, 2.0, 17, 9, "cuda")
    exact = O.scaling_bias(O.amax(OS.f64_to_bf16(OS.swiglu_backward(OS.bf16_to_f64(ref.bf16), bits_of(y_pre)))), O.E5, conv)
    w8, w8t = (None, qw.y_t) if layout == "t" else (qw.y, None)
    for bias, clip in ((exact, None), (exact + 2, True), (exact - 4, False)):
        dz = torch.full((T, F), float("nan"), dtype=torch.bfloat16, device="cuda")
        gg = torch.full((T, 2 * F), float("nan"), dtype=torch.bfloat16, device="cuda")
        g8 = torch.full((T, 2 * F), 0xAA, dtype=torch.uint8, device="cuda")
        amax_g = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        ctx.linear_dgrad_q(qg.y, qg.bias, w8, w8t, qw.bias, g8, _dev_i32(bias), y_pre=y_pre, dx=dz, g=gg,
                           d_amax_g=amax_g, act=lib.ACT_SWIGLU, conv=conv)
        assert_bf16_within_one_ulp(bits_of(dz), ref)
        want = OS.f64_to_bf16(OS.swiglu_backward(OS.bf16_to_f64(bits_of(dz)), bits_of(y_pre)))
        d = np.abs(bf16_ordinal(bits_of(gg)) - bf16_ordinal(want))
        assert d.max() <= 1, d.max()
        _check_bytes(ctx, lib, gg, g8, amax_g, bias, O.E5, conv, clip)
    gg2 = torch.full((T, 2 * F), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.linear_dgrad_act(qg.y, qg.bias, w8, w8t, qw.bias, y_pre, None, gg2, act=lib.ACT_SWIGLU, conv=conv)
    assert torch.equal(gg2, gg)
    assert ctx.device_flags(clear=True) == 0


def test_swiglu_argument_errors(ctx, lib):
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    x8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    w8 = torch.zeros((96, 64), dtype=torch.uint8, device="cuda")            # N = 96 is not a multiple of 64
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_q(x8, b, w8, b, torch.zeros((32, 48), dtype=torch.uint8, device="cuda"), b, act=lib.ACT_SWIGLU)
    assert e.value.status == lib.ERR_ALIGN
    dy8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    wd = torch.zeros((64, 48), dtype=torch.uint8, device="cuda")            # K = 48 is not a multiple of 32
    pre = torch.zeros((32, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad_q(dy8, b, wd, None, b, torch.zeros((32, 96), dtype=torch.uint8, device="cuda"), b, y_pre=pre,
                           act=lib.ACT_SWIGLU)
    assert e.value.status == lib.ERR_ALIGN
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad_q(dy8, b, torch.zeros((64, 64), dtype=torch.uint8, device="cuda"), None, b,
                           torch.zeros((32, 128), dtype=torch.uint8, device="cuda"), b, act=lib.ACT_SWIGLU)  # no y_pre
    assert e.value.status == lib.ERR_NULL
    assert ctx.device_flags(clear=True) == 0


def test_llama_mlp_block_forward_and_backward_chain(ctx, lib):
    """gate_up (SwiGLU epilogue, FP8 bytes out) -> down -> dY -> down's input gradient (SwiGLU backward epilogue,
    E5 bytes out) -> gate_up's weight and input gradients, all on bytes the epilogues wrote; every matmul is
    checked against the oracle fed the GPU's own operand bytes, and the interleaved layouts must line up (the
    gradient bytes [T, 2F] against the interleaved weight [2F, K])."""
    conv = O.CONV_PAPER
    T, K, F = 320, 256, 160
    x = I.normal_bf16(T, K, 1.0, 91, 1, "cuda")
    qx = Quantised(ctx, x, O.E4, conv)
    qgu = _interleaved_weight(ctx, F, K, conv, 92)
    qd = Quantised(ctx, I.normal_bf16(K, F, 0.05, 93, 2, "cuda"), O.E4, conv)      # down: F -> K
    dev = dict(device="cuda")
    y_pre = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)
    z = torch.empty((T, F), dtype=torch.bfloat16, **dev)
    z8 = torch.empty((T, F), dtype=torch.uint8, **dev)
    amax_z = torch.zeros(1, dtype=torch.float32, **dev)
    bz = _dev_i32(4)
    ctx.linear_fwd_q(qx.y, qx.bias, qgu.y, qgu.bias, z8, bz, y_pre=y_pre, z=z, d_amax_z=amax_z, act=lib.ACT_SWIGLU)
    assert_codes_equal(u8(z8), O.cast(bits_of(z), 4 + 1, O.N_E4), O.N_E4)
    out = torch.empty((T, K), dtype=torch.bfloat16, **dev)
    ctx.linear_fwd(z8, bz, qd.y, qd.bias, out)
    assert_bf16_within_one_ulp(bits_of(out), O.linear_fwd_np(u8(z8), 4 + 1, qd.ref, qd.shift))
    # backward from a seeded output gradient
    qdy = Quantised(ctx, I.normal_bf16(T, K, 1e-3, 94, 3, "cuda"), O.E5, conv)
    g = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)
    g8 = torch.empty((T, 2 * F), dtype=torch.uint8, **dev)
    dz = torch.empty((T, F), dtype=torch.bfloat16, **dev)
    amax_g = torch.zeros(1, dtype=torch.float32, **dev)
    dz_ref = O.linear_dgrad_np(qdy.ref, qdy.shift, qd.ref, qd.shift)
    bq = O.scaling_bias(O.amax(OS.f64_to_bf16(OS.swiglu_backward(OS.bf16_to_f64(dz_ref.bf16), bits_of(y_pre)))), O.E5) - 1
    ctx.linear_dgrad_q(qdy.y, qdy.bias, qd.y, None, qd.bias, g8, _dev_i32(bq), y_pre=y_pre, dx=dz, g=g, d_amax_g=amax_g,
                       act=lib.ACT_SWIGLU)
    assert_bf16_within_one_ulp(bits_of(dz), dz_ref)
    assert_codes_equal(u8(g8), O.cast(bits_of(g), bq, O.N_E5), O.N_E5)
    # gate_up's gradients from those bytes: dW[2F, K] keeps the weight's row layout, dX[T, K]
    dw = torch.empty((2 * F, K), dtype=torch.bfloat16, **dev)
    dx = torch.empty((T, K), dtype=torch.bfloat16, **dev)
    bqt = _dev_i32(bq)
    ctx.linear_wgrad(g8, None, bqt, qx.y, None, qx.bias, dw, T)
    ctx.linear_dgrad(g8, bqt, qgu.y, None, qgu.bias, dx)
    assert_bf16_within_one_ulp(bits_of(dw), O.linear_wgrad_np(u8(g8), bq, qx.ref, qx.shift))
    assert_bf16_within_one_ulp(bits_of(dx), O.linear_dgrad_np(u8(g8), bq, qgu.ref, qgu.shift))
    assert ctx.device_flags(clear=True) & ~lib.FLAG_SATURATED == 0


def test_llama7b_gate_up_with_swiglu_at_benchmark_size_sampled(ctx, lib):
    """The Llama-2-7B gate_up layer (8192 tokens, 4096 -> 2 x 11008) in the benchmark's launch configuration with the
    SwiGLU epilogue: pre-activations at sampled positions against the oracle, z and its bytes as relations on the
    GPU's own stored tensors at the same positions, the amax against a reduction over the whole of z."""
    T, K, F = 8192, 4096, 11008
    x = I.normal_bf16(T, K, 1.0, 8100, 1, "cuda", outlier_frac=0.005, outlier_scale=100.0)
    qx = Quantised(ctx, x, O.E4, O.CONV_PAPER)
    qw = _interleaved_weight(ctx, F, K, O.CONV_PAPER, 8101)
    y_pre = torch.empty((T, 2 * F), dtype=torch.bfloat16, device="cuda")
    z = torch.empty((T, F), dtype=torch.bfloat16, device="cuda")
    z8 = torch.empty((T, F), dtype=torch.uint8, device="cuda")
    amax_z = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = 1
    ctx.linear_fwd_q(qx.y, qx.bias, qw.y, qw.bias, z8, _dev_i32(bias), y_pre=y_pre, z=z, d_amax_z=amax_z,
                     act=lib.ACT_SWIGLU)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    rng = np.random.default_rng(81)
    rows = np.concatenate([rng.integers(0, T, 3000), [0, T - 1, 0, T - 1]])
    feat = np.concatenate([rng.integers(0, F, 3000), [0, F - 1, F - 1, 0]])
    gi, ui = OS._blocks32(2 * F)
    r_t = torch.from_numpy(rows).cuda()
    for cols in (gi[feat], ui[feat]):
        ref = O.linear_samples(O.FWD, qx.ref, O.N_E4, qx.shift, qw.ref, O.N_E4, qw.shift, rows, cols)
        got = y_pre[r_t, torch.from_numpy(cols).cuda()]
        assert_bf16_within_one_ulp(bits_of(got.reshape(1, -1))[0], ref)
    g = OS.bf16_to_f64(bits_of(y_pre[r_t, torch.from_numpy(gi[feat]).cuda()].reshape(1, -1)))
    u = OS.bf16_to_f64(bits_of(y_pre[r_t, torch.from_numpy(ui[feat]).cuda()].reshape(1, -1)))
    want = OS.f64_to_bf16(OS.silu(g) * u)
    zs = z[r_t, torch.from_numpy(feat).cuda()].reshape(1, -1)
    assert np.abs(bf16_ordinal(bits_of(zs)) - bf16_ordinal(want)).max() <= 1
    z8s = z8[r_t, torch.from_numpy(feat).cuda()].reshape(1, -1)
    assert_codes_equal(u8(z8s), O.cast(bits_of(zs), bias + 1, O.N_E4), O.N_E4)
    assert float(amax_z.item()) == float(z.float().abs().max().item())


def test_llama7b_down_input_gradient_with_swiglu_backward_at_benchmark_size_sampled(ctx, lib):
    """The backward twin at benchmark size: dz[8192, 11008] = dY8 . W8 (contraction 4096, weight read in its forward
    layout) with the SwiGLU backward epilogue producing the [8192, 22016] gate / up gradient, its E5 bytes and amax."""
    T, N, F = 8192, 4096, 11008
    qg = Quantised(ctx, I.normal_bf16(T, N, 1e-5, 8200, 3, "cuda"), O.E5, O.CONV_PAPER)
    qw = Quantised(ctx, I.normal_bf16(N, F, 0.02, 8201, 2, "cuda"), O.E4, O.CONV_PAPER)
    y_pre = I.normal_bf16(T, 2 * F, 1.5, 8202, 9, "cuda")
    dz = torch.empty((T, F), dtype=torch.bfloat16, device="cuda")
    g = torch.empty((T, 2 * F), dtype=torch.bfloat16, device="cuda")
    g8 = torch.empty((T, 2 * F), dtype=torch.uint8, device="cuda")
    amax_g = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = 28
    ctx.linear_dgrad_q(qg.y, qg.bias, qw.y, None, qw.bias, g8, _dev_i32(bias), y_pre=y_pre, dx=dz, g=g, d_amax_g=amax_g,
                       act=lib.ACT_SWIGLU)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    rng = np.random.default_rng(82)
    rows = np.concatenate([rng.integers(0, T, 3000), [0, T - 1, 0, T - 1]])
    feat = np.concatenate([rng.integers(0, F, 3000), [0, F - 1, F - 1, 0]])
    r_t, f_t = torch.from_numpy(rows).cuda(), torch.from_numpy(feat).cuda()
    ref = O.linear_samples(O.DGRAD, qg.ref, O.N_E5, qg.shift, qw.ref, O.N_E4, qw.shift, rows, feat)
    dzs = dz[r_t, f_t].reshape(1, -1)
    assert_bf16_within_one_ulp(bits_of(dzs)[0], ref)
    gi, ui = OS._blocks32(2 * F)
    gcol, ucol = torch.from_numpy(gi[feat]).cuda(), torch.from_numpy(ui[feat]).cuda()
    a = OS.bf16_to_f64(bits_of(y_pre[r_t, gcol].reshape(1, -1)))
    u = OS.bf16_to_f64(bits_of(y_pre[r_t, ucol].reshape(1, -1)))
    d = OS.bf16_to_f64(bits_of(dzs))
    e = np.exp(-np.abs(a))
    s = np.where(a > 0, 1.0 / (1.0 + e), e / (1.0 + e))
    for cols, want in ((gcol, d * u * (s + a * s * (1.0 - s))), (ucol, d * OS.silu(a))):
        got = g[r_t, cols].reshape(1, -1)
        assert np.abs(bf16_ordinal(bits_of(got)) - bf16_ordinal(OS.f64_to_bf16(want))).max() <= 1
        assert_codes_equal(u8(g8[r_t, cols].reshape(1, -1)), O.cast(bits_of(got), bias, O.N_E5), O.N_E5)
    assert float(amax_g.item()) == float(g.float().abs().max().item())
