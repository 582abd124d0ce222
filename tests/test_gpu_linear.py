"""GPU parity: the three FP8 matmuls with unscale against the CPU oracle.

Both sides start from the same seeded bf16 tensors.  The FP8 bytes and biases
must agree bit for bit; FP32 outputs must lie within 2^-14 * sum_k |a*b| of
the exact value; bf16 outputs within one bf16 ulp of the oracle's rounding.
"""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import (assert_bf16_within_one_ulp, assert_codes_equal, assert_gemm_close, bits_of, tile_sample_positions,
                     u8)
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


class Quantised:
    """One tensor quantised on the GPU (both layouts) and by the oracle."""

    def __init__(self, ctx, x, kind, conv, margin=0, transposed=True):
        """transposed=False asks for the row-major bytes only, which is what the benchmark's steps do."""
        rows, cols = x.shape
        self.kind, self.conv = kind, conv
        self.amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.y = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
        self.y_t = torch.empty((cols, rows), dtype=torch.uint8, device="cuda") if transposed else None
        cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
        cast(x, None, conv=conv, margin=margin, d_amax_out=self.amax, d_bias_out=self.bias, y=self.y, y_t=self.y_t)
        a, b, ref = O.quantise(bits_of(x), kind, conv, margin)
        assert float(self.amax.item()) == a and int(self.bias.item()) == b
        fmt = O.native_format(kind)
        assert_codes_equal(u8(self.y), ref, fmt)
        if transposed:
            assert_codes_equal(u8(self.y_t), np.ascontiguousarray(ref.T), fmt)
        self.ref, self.ref_bias, self.shift = ref, b, b + O.delta(kind, conv)


def _layer(ctx, T, K, N, conv, seed, x_std=1.0, w_std=0.02, g_std=1e-3, margin=0):
    x = I.normal_bf16(T, K, x_std, seed, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0)
    w = I.normal_bf16(N, K, w_std, seed, 2, "cuda")
    g = I.normal_bf16(T, N, g_std, seed, 3, "cuda")
    return (Quantised(ctx, x, O.E4, conv), Quantised(ctx, w, O.E4, conv), Quantised(ctx, g, O.E5, conv, margin))


SHAPES = [
    (272, 8208, 304),    # few tiles of the CTA-pair kernel, long ragged contraction: sliced, partial sums, finalize
    (256, 768, 768),     # config 1
    (128, 128, 256),     # exactly one tile, one k-block
    (128, 16, 256),      # shortest contraction the API allows
    (144, 272, 528),     # ragged in every dimension (multiples of 16 where the layout needs it)
    (400, 1040, 784),    # several tiles, several k-blocks, ragged tails
    (16, 2048, 48),      # skinny
]


@pytest.mark.parametrize("T,K,N", SHAPES)
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_fwd_dgrad_wgrad_match_oracle(ctx, lib, T, K, N, conv):
    qx, qw, qg = _layer(ctx, T, K, N, conv, seed=T * 1000003 + K * 101 + N)
    for dt in (torch.float32, torch.bfloat16):
        y = torch.full((T, N), float("nan"), dtype=dt, device="cuda")
        dx = torch.full((T, K), float("nan"), dtype=dt, device="cuda")
        dw = torch.full((N, K), float("nan"), dtype=dt, device="cuda")
        # backward operands either as transposed copies (contraction over contiguous bytes) or in the forward
        # layout (contraction strided), and mixed
        dx2 = torch.full((T, K), float("nan"), dtype=dt, device="cuda")
        dw2 = torch.full((N, K), float("nan"), dtype=dt, device="cuda")
        dw3 = torch.full((N, K), float("nan"), dtype=dt, device="cuda")
        ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y, conv=conv)
        ctx.linear_dgrad(qg.y, qg.bias, None, qw.y_t, qw.bias, dx, conv=conv)
        ctx.linear_wgrad(None, qg.y_t, qg.bias, None, qx.y_t, qx.bias, dw, T, conv=conv)
        ctx.linear_dgrad(qg.y, qg.bias, qw.y, None, qw.bias, dx2, conv=conv)
        ctx.linear_wgrad(qg.y, None, qg.bias, qx.y, None, qx.bias, dw2, T, conv=conv)
        ctx.linear_wgrad(qg.y, None, qg.bias, None, qx.y_t, qx.bias, dw3, T, conv=conv)
        assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
        refs = (O.linear_fwd(qx.ref, qx.shift, qw.ref, qw.shift),
                O.linear_dgrad(qg.ref, qg.shift, qw.ref, qw.shift),
                O.linear_wgrad(qg.ref, qg.shift, qx.ref, qx.shift))
        refs = refs + (refs[1], refs[2], refs[2])
        for got, ref in zip((y, dx, dw, dx2, dw2, dw3), refs):
            if dt == torch.float32:
                worst = assert_gemm_close(got.cpu().numpy(), ref)
                print(f"[parity] T={T} K={K} N={N} conv={conv}: max |err| / sum|a*b| = 2^{np.log2(max(worst, 1e-300)):.1f}")
            else:
                assert_bf16_within_one_ulp(bits_of(got), ref)


def test_fwd_bias_vector_and_output_amax(ctx, lib):
    T, K, N = 200, 512, 300
    qx, qw, _ = _layer(ctx, T, K, N + 4, O.CONV_PAPER, seed=99)
    w8 = qw.y[:N].contiguous()
    for bias_dt in (torch.bfloat16, torch.float32):
        bv = (torch.randn(N, device="cuda") * 0.5).to(bias_dt)
        ref = O.linear_fwd(qx.ref, qx.shift, qw.ref[:N], qw.shift, bias_vec=bv.double().cpu().numpy())
        for dt in (torch.float32, torch.bfloat16):
            y = torch.empty((T, N), dtype=dt, device="cuda")
            amax_y = torch.full((1,), 123.0, dtype=torch.float32, device="cuda")
            ctx.linear_fwd(qx.y, qx.bias, w8, qw.bias, y, bias_vec=bv, d_amax_y=amax_y)
            if dt == torch.float32:
                assert_gemm_close(y.cpu().numpy(), ref)
            else:
                assert_bf16_within_one_ulp(bits_of(y), ref)
            # the emitted amax is exactly the amax of what was written
            assert float(amax_y.item()) == float(y.float().abs().max().item())


@pytest.mark.parametrize("T,K,N", [(256, 768, 768), (144, 272, 528), (64, 1024, 512), (400, 1040, 784)])
def test_fwd_with_gelu_in_the_epilogue(ctx, lib, T, K, N):
    """The pre-activation must meet the forward bar; the activated tensor must be GELU of exactly that
    pre-activation (checked with the float64 GELU on the GPU's own pre-activation bits: a relation between two
    outputs of the call, not an expected value), and the emitted amax must be the amax of what was written."""
    from oracle import stack as OS
    from helpers import bf16_ordinal
    qx, qw, _ = _layer(ctx, T, K, N, O.CONV_PAPER, seed=4242 + T)
    bv = (torch.randn(N, device="cuda") * 0.3).to(torch.bfloat16)
    ref = O.linear_fwd_np(qx.ref, qx.shift, qw.ref, qw.shift, bias_vec=bv.double().cpu().numpy())
    for want_pre in (True, False):
        y_pre = torch.full((T, N), float("nan"), dtype=torch.bfloat16, device="cuda") if want_pre else None
        y_act = torch.full((T, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        amax_act = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        ctx.linear_fwd_act(qx.y, qx.bias, qw.y, qw.bias, y_pre, y_act, bias_vec=bv, d_amax_act=amax_act)
        assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
        if want_pre:
            assert_bf16_within_one_ulp(bits_of(y_pre), ref)
            gelu_of_pre = OS.gelu_bits(bits_of(y_pre))
            d = np.abs(bf16_ordinal(bits_of(y_act)) - bf16_ordinal(gelu_of_pre))
            assert d.max() <= 1, d.max()
            kept = bits_of(y_act)
        else:
            assert np.array_equal(bits_of(y_act), kept)   # same activated tensor with or without the first output
        assert float(amax_act.item()) == float(y_act.float().abs().max().item())


@pytest.mark.parametrize("T,K,N", [(256, 768, 768), (144, 272, 528), (64, 1024, 512), (400, 1040, 784)])
def test_dgrad_with_gelu_backward_in_the_epilogue(ctx, lib, T, K, N):
    """dX must meet the input-gradient bar; the second output must be bf16(dX) * GELU'(y_pre) (checked in float64
    on the GPU's own dX bits and the given pre-activation), and the emitted amax the amax of what was written."""
    from oracle import stack as OS
    from helpers import bf16_ordinal
    qx, qw, qg = _layer(ctx, T, K, N, O.CONV_PAPER, seed=777 + T)
    y_pre = I.normal_bf16(T, K, 1.5, 11, 9, "cuda")
    ref = O.linear_dgrad_np(qg.ref, qg.shift, qw.ref, qw.shift)
    for want_dx, layout in ((True, "t"), (False, "t"), (True, "mn")):
        dx = torch.full((T, K), float("nan"), dtype=torch.bfloat16, device="cuda") if want_dx else None
        g = torch.full((T, K), float("nan"), dtype=torch.bfloat16, device="cuda")
        amax_g = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        w8, w8t = (None, qw.y_t) if layout == "t" else (qw.y, None)
        ctx.linear_dgrad_act(qg.y, qg.bias, w8, w8t, qw.bias, y_pre, dx, g, d_amax_act=amax_g)
        assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
        if want_dx:
            assert_bf16_within_one_ulp(bits_of(dx), ref)
            want = OS.f64_to_bf16(OS.bf16_to_f64(bits_of(dx)) * OS.gelu_grad(bits_of(y_pre)))
            d = np.abs(bf16_ordinal(bits_of(g)) - bf16_ordinal(want))
            assert d.max() <= 1, d.max()
            kept = bits_of(g)
        else:
            assert np.array_equal(bits_of(g), kept)
        assert float(amax_g.item()) == float(g.float().abs().max().item())


def test_dgrad_amax_and_margin(ctx, lib):
    T, K, N = 256, 384, 512
    qx, qw, qg = _layer(ctx, T, K, N, O.CONV_PAPER, seed=5, margin=3)
    dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    amax_dx = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.linear_dgrad(qg.y, qg.bias, None, qw.y_t, qw.bias, dx, d_amax_dx=amax_dx)
    assert_bf16_within_one_ulp(bits_of(dx), O.linear_dgrad(qg.ref, qg.shift, qw.ref, qw.shift))
    assert float(amax_dx.item()) == float(dx.float().abs().max().item())


def test_extreme_biases_unscale_exactly(ctx, lib):
    """Tensors near the ends of the bf16 range: biases beyond +-126 need the
    two-step power-of-two unscale."""
    T, K, N = 128, 64, 256
    x = I.normal_bf16(T, K, 2.0 ** -120, 7, 1, "cuda")
    w = I.normal_bf16(N, K, 2.0 ** 100, 7, 2, "cuda")
    qx, qw = Quantised(ctx, x, O.E4, O.CONV_PAPER), Quantised(ctx, w, O.E4, O.CONV_PAPER)
    assert qx.ref_bias > 110 and qw.ref_bias < -90
    y = torch.empty((T, N), dtype=torch.float32, device="cuda")
    ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y)
    assert_gemm_close(y.cpu().numpy(), O.linear_fwd(qx.ref, qx.shift, qw.ref, qw.shift))
    tiny = I.normal_bf16(T, K, 2.0 ** -125, 7, 4, "cuda")
    qt = Quantised(ctx, tiny, O.E4, O.CONV_PAPER)
    # tiny x tiny: the unscale exponent is beyond -126 and the result underflows FP32
    out = torch.empty((T, T), dtype=torch.float32, device="cuda")
    ctx.linear_fwd(qt.y, qt.bias, qx.y, qx.bias, out)
    assert_gemm_close(out.cpu().numpy(), O.linear_fwd(qt.ref, qt.shift, qx.ref, qx.shift))


def test_matmul_argument_errors(ctx, lib):
    x8 = torch.zeros((32, 24), dtype=torch.uint8, device="cuda")   # K = 24 is not a multiple of 16
    w8 = torch.zeros((64, 24), dtype=torch.uint8, device="cuda")
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.zeros((32, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd(x8, b, w8, b, y)
    assert e.value.status == lib.ERR_ALIGN
    g8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    dx = torch.zeros((32, 32), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad(g8, b, w8[:, :8].contiguous(), None, b, dx[:, :8].contiguous())   # K = 8: rows of W8 not 16-byte multiples
    assert e.value.status == lib.ERR_ALIGN
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad(g8, b, None, None, b, dx)
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd(x8, None, w8, b, y)
    assert e.value.status == lib.ERR_NULL


@pytest.mark.parametrize("wl_name,layer", [("c2_gpt", 0), ("c2_gpt", 1), ("c2_gpt", 2), ("c2_gpt", 3),
                                           ("c3_llama7b", 0), ("c3_llama7b", 1), ("c3_llama7b", 2), ("c3_llama7b", 3)])
def test_full_size_layers_sampled(ctx, lib, wl_name, layer):
    """Every layer of the GPT block and of the Llama-2-7B block at benchmark size, in the benchmark's launch
    configuration (forward layouts, no transposed copies): bytes and biases checked in full; each matmul output
    at 64 positions in every 128 x 128 block, on eight whole blocks and on its first / last rows and columns."""
    wl = I.WORKLOADS[wl_name]
    l = wl.layers[layer]
    T, K, N = wl.tokens, l.K, l.N
    t = I.layer_tensors(wl, layer, device="cuda")
    qx = Quantised(ctx, t["x"], O.E4, O.CONV_PAPER, transposed=False)
    qw = Quantised(ctx, t["w"], O.E4, O.CONV_PAPER, transposed=False)
    qg = Quantised(ctx, t["g"], O.E5, O.CONV_PAPER, transposed=False)
    del t
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y)
    ctx.linear_dgrad(qg.y, qg.bias, qw.y, None, qw.bias, dx)
    ctx.linear_wgrad(qg.y, None, qg.bias, qx.y, None, qx.bias, dw, T)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    rng = np.random.default_rng(layer + 1)
    cases = ((O.FWD, y, (qx.ref, O.N_E4, qx.shift, qw.ref, O.N_E4, qw.shift)),
             (O.DGRAD, dx, (qg.ref, O.N_E5, qg.shift, qw.ref, O.N_E4, qw.shift)),
             (O.WGRAD, dw, (qg.ref, O.N_E5, qg.shift, qx.ref, O.N_E4, qx.shift)))
    for kind, out, ops in cases:
        rows, cols = tile_sample_positions(rng, out.shape[0], out.shape[1])
        ref = O.linear_samples(kind, *ops, rows, cols)
        got = bits_of(out)[rows, cols]
        frac = assert_bf16_within_one_ulp(got, ref)
        print(f"[parity] {wl_name}/{l.name} kind {kind}: {rows.size} positions, {frac:.5f} through the cancellation branch")


@pytest.mark.parametrize("T,K,N", [(256, 768, 768), (400, 1040, 784), (16, 4096, 1280), (3, 16384, 272), (272, 8208, 304)])
def test_bf16_output_is_the_rounded_fp32_output(ctx, lib, T, K, N):
    """The bf16 result of a call equals the FP32 result of the same call on the same operands rounded to bf16
    (nearest even), bit for bit: the two output types differ in the last step of the epilogue only.  Covers the
    CTA-pair kernel, the single-CTA kernel and the split contraction with its finishing kernel."""
    qx, qw, qg = _layer(ctx, T, K, N, O.CONV_PAPER, seed=31337 + T)
    calls = (lambda out: ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, out), (T, N)), \
            (lambda out: ctx.linear_dgrad(qg.y, qg.bias, qw.y, None, qw.bias, out), (T, K)), \
            (lambda out: ctx.linear_wgrad(qg.y, None, qg.bias, qx.y, None, qx.bias, out, T), (N, K))
    for call, shape in calls:
        o32 = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        o16 = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        call(o32)
        call(o16)
        assert np.array_equal(bits_of(o16), O.f32_to_bf16_bits_np(o32.cpu().numpy()))
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


@pytest.mark.parametrize("T,K,N", [(1, 2048, 768), (16, 4096, 1280), (64, 8192, 512), (100, 1024, 2304),
                                   (5, 2064, 784), (128, 4096, 4096), (3, 16384, 272), (33, 1024, 18944), (9, 2048, 786)])
def test_decode_shapes_split_k(ctx, lib, T, K, N):
    """Few tokens, long contraction: the library deals the k-blocks of all output
    tiles evenly to the SMs and finishes in a second kernel; results must meet
    the same bars (ragged last k-block, ragged last tile, tiles cut in two and
    in many pieces included)."""
    x = I.normal_bf16(T, K, 1.0, 31, 1, "cuda", outlier_frac=0.005, outlier_scale=100.0)
    w = I.normal_bf16(N, K, 0.015, 31, 2, "cuda")
    qx, qw = Quantised(ctx, x, O.E4, O.CONV_PAPER), Quantised(ctx, w, O.E4, O.CONV_PAPER)
    ref = O.linear_fwd(qx.ref, qx.shift, qw.ref, qw.shift)
    bv = (torch.randn(N, device="cuda") * 0.1).to(torch.bfloat16)
    ref_b = O.linear_fwd(qx.ref, qx.shift, qw.ref, qw.shift, bias_vec=bv.double().cpu().numpy())
    for dt in (torch.float32, torch.bfloat16):
        y = torch.full((T, N), float("nan"), dtype=dt, device="cuda")
        amax_y = torch.zeros(1, dtype=torch.float32, device="cuda")
        ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y, d_amax_y=amax_y)
        if dt == torch.float32:
            assert_gemm_close(y.cpu().numpy(), ref)
        else:
            assert_bf16_within_one_ulp(bits_of(y), ref)
        assert float(amax_y.item()) == float(y.float().abs().max().item())
        ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y, bias_vec=bv)
        if dt == torch.float32:
            assert_gemm_close(y.cpu().numpy(), ref_b)
        else:
            assert_bf16_within_one_ulp(bits_of(y), ref_b)
        # the inference call (weights final long before: it may read them early) gives the same bits
        y2 = torch.full((T, N), float("nan"), dtype=dt, device="cuda")
        ctx.linear_infer(qx.y, qx.bias, qw.y, qw.bias, y2, bias_vec=bv)
        assert torch.equal(y.view(torch.int16 if dt == torch.bfloat16 else torch.int32),
                           y2.view(torch.int16 if dt == torch.bfloat16 else torch.int32))
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def _infer_cast(ctx, x, w8, d_bw, dt, conv=O.CONV_PAPER, margin=0, bias_vec=None):
    """fp8_linear_infer_cast on fresh outputs (poisoned first): amax, bias, bytes of x and the product."""
    T, K = x.shape
    x8 = torch.full((T, K), 0x55, dtype=torch.uint8, device="cuda")
    amax = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    bias = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    y = torch.full((T, w8.shape[0]), float("nan"), dtype=dt, device="cuda")
    amax_y = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.linear_infer_cast(x, amax, bias, x8, w8, d_bw, y, margin=margin, bias_vec=bias_vec, d_amax_y=amax_y, conv=conv)
    return x8, amax, bias, y, amax_y


@pytest.mark.parametrize("T,K,N", [(1, 2048, 768), (1, 28672, 1024), (4, 8192, 1280), (3, 1024, 272), (2, 16384, 512),
                                   (5, 2064, 784), (16, 4096, 1280), (64, 8192, 512), (128, 4096, 4096), (33, 1024, 18944)])
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_inference_call_that_quantises_its_activation(ctx, lib, T, K, N, conv):
    """fp8_linear_infer_cast: one call for FP8-AMAX of the activation and the forward matmul (Section 3.1).  amax,
    bias and bytes of x must be the oracle's bit for bit, the product must meet the forward bars and carry the same
    bits as fp8_cast_e4 followed by fp8_linear_infer, both for activations small enough for the single launch
    (at most 64 KB) and for larger ones."""
    x = I.normal_bf16(T, K, 1.0, 53, 1, "cuda", outlier_frac=0.005, outlier_scale=100.0)
    w = I.normal_bf16(N, K, 0.015, 53, 2, "cuda")
    qx, qw = Quantised(ctx, x, O.E4, conv, transposed=False), Quantised(ctx, w, O.E4, conv, transposed=False)
    bv = (torch.randn(N, device="cuda") * 0.1).to(torch.bfloat16)
    ref = O.linear_fwd(qx.ref, qx.shift, qw.ref, qw.shift, bias_vec=bv.double().cpu().numpy())
    for dt in (torch.float32, torch.bfloat16):
        for _ in range(2):   # a second call finds the context's scratch as the first left it
            x8, amax, bias, y, amax_y = _infer_cast(ctx, x, qw.y, qw.bias, dt, conv=conv, bias_vec=bv)
            assert float(amax.item()) == float(qx.amax.item()) and int(bias.item()) == qx.ref_bias
            assert_codes_equal(u8(x8), qx.ref, O.N_E4)
            if dt == torch.float32:
                assert_gemm_close(y.cpu().numpy(), ref)
            else:
                assert_bf16_within_one_ulp(bits_of(y), ref)
            assert float(amax_y.item()) == float(y.float().abs().max().item())
            y2 = torch.full((T, N), float("nan"), dtype=dt, device="cuda")
            ctx.linear_infer(qx.y, qx.bias, qw.y, qw.bias, y2, bias_vec=bv, conv=conv)
            as_int = torch.int16 if dt == torch.bfloat16 else torch.int32
            assert torch.equal(y.view(as_int), y2.view(as_int))
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_inference_call_margin_specials_and_other_input_types(ctx, lib):
    """The margin of Section 3.2 reaches the bias; an all-zero activation gives bias 0 and the ZERO_AMAX flag as
    fp8_cast_e4 does; FP16 / FP32 activations and unaligned ones take the two-call route with the same results."""
    T, K, N = 2, 4096, 512
    w = I.normal_bf16(N, K, 0.02, 59, 2, "cuda")
    qw = Quantised(ctx, w, O.E4, O.CONV_PAPER, transposed=False)
    x = I.normal_bf16(T, K, 3.0, 59, 1, "cuda")
    a, b, ref8 = O.quantise(bits_of(x), O.E4, O.CONV_PAPER, 3)
    x8, amax, bias, y, _ = _infer_cast(ctx, x, qw.y, qw.bias, torch.float32, margin=3)
    assert float(amax.item()) == a and int(bias.item()) == b
    assert_codes_equal(u8(x8), ref8, O.N_E4)
    assert_gemm_close(y.cpu().numpy(), O.linear_fwd(ref8, b + 1, qw.ref, qw.shift))
    ctx.device_flags(clear=True)
    z = torch.zeros((T, K), dtype=torch.bfloat16, device="cuda")
    x8, amax, bias, y, _ = _infer_cast(ctx, z, qw.y, qw.bias, torch.float32)
    assert float(amax.item()) == 0.0 and int(bias.item()) == 0 and not x8.any() and not y.any()
    assert ctx.device_flags(clear=True) & lib.FLAG_ZERO_AMAX
    for xin in (x.to(torch.float16), x.float(), torch.cat([x.flatten()[:1], x.flatten()])[1:].view(T, K)):
        a, b, ref8 = O.quantise(bits_of(xin.to(torch.bfloat16)), O.E4) if xin.dtype == torch.bfloat16 else (None, None, None)
        x8, amax, bias, y, _ = _infer_cast(ctx, xin, qw.y, qw.bias, torch.bfloat16)
        x8b = torch.empty_like(x8)
        amax_b, bias_b = torch.zeros_like(amax), torch.zeros_like(bias)
        ctx.cast_e4(xin, None, d_amax_out=amax_b, d_bias_out=bias_b, y=x8b)
        y_b = torch.empty_like(y)
        ctx.linear_infer(x8b, bias_b, qw.y, qw.bias, y_b)
        assert torch.equal(x8, x8b) and torch.equal(amax, amax_b) and torch.equal(bias, bias_b)
        assert torch.equal(y.view(torch.int16), y_b.view(torch.int16))
        if ref8 is not None:
            assert_codes_equal(u8(x8), ref8, O.N_E4)
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_infer_cast(x, amax, None, x8, qw.y, qw.bias, y)
    assert e.value.status == lib.ERR_NULL
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


@pytest.mark.parametrize("T,K,N", [(256, 768, 768), (2048, 1024, 1024), (16, 4096, 1280), (1, 8192, 1024), (1, 28672, 1024)])
def test_calls_chained_without_host_synchronisation_see_each_others_results(ctx, lib, T, K, N):
    """Inside a step the library's kernels follow each other as programmatic dependent launches: a kernel is resident
    while the one before it still runs and must not read a bias before that one has written it.  Quantise and multiply
    back to back with no host synchronisation in between, the bias words and bytes poisoned before every round, through
    each quantisation route (two launches, one pass with a wrong guess, the grouped call in both modes); every round
    must give the bits of a run that synchronises between the calls."""
    x = I.normal_bf16(T, K, 1.0, 61, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0)
    w = I.normal_bf16(N, K, 0.02, 61, 2, "cuda")
    qx, qw = Quantised(ctx, x, O.E4, O.CONV_PAPER, transposed=False), Quantised(ctx, w, O.E4, O.CONV_PAPER, transposed=False)
    y_ref = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ctx.linear_fwd(qx.y, qx.bias, qw.y, qw.bias, y_ref)
    torch.cuda.synchronize()
    x8, w8 = torch.empty_like(qx.y), torch.empty_like(qw.y)
    amax = torch.zeros(2, dtype=torch.float32, device="cuda")
    bias = torch.zeros(2, dtype=torch.int32, device="cuda")
    y = torch.empty_like(y_ref)

    def two_launches():
        ctx.cast_e4(w, None, d_amax_out=amax[0:1], d_bias_out=bias[0:1], y=w8)
        ctx.cast_e4(x, None, d_amax_out=amax[1:2], d_bias_out=bias[1:2], y=x8)

    def one_pass_wrong_guess():
        ctx.cast_predicted(lib.E4, w, amax[0:1], bias[0:1], w8)
        ctx.cast_predicted(lib.E4, x, amax[1:2], bias[1:2], x8)

    items = [(lib.E4, w, amax[0:1], bias[0:1], w8), (lib.E4, x, amax[1:2], bias[1:2], x8)]
    routes = (two_launches, one_pass_wrong_guess, lambda: ctx.cast_group(items), lambda: ctx.cast_group(items, predicted=True))
    for route in routes:
        for rnd in range(12):
            bias.fill_(60 + rnd)     # an absurd bias: a matmul that read it would be off by dozens of powers of two
            x8.fill_(0x55)
            w8.fill_(0x55)
            y.fill_(float("nan"))
            route()
            ctx.linear_fwd(x8, bias[1:2], w8, bias[0:1], y)
            torch.cuda.synchronize()
            assert int(bias[0].item()) == qw.ref_bias and int(bias[1].item()) == qx.ref_bias
            assert torch.equal(x8, qx.y) and torch.equal(w8, qw.y)
            assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)), f"round {rnd}"
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


@pytest.mark.parametrize("T,N,K", [(16, 4096, 1024), (2, 8208, 528)])
def test_decode_shapes_dgrad_from_row_major_weights(ctx, lib, T, N, K):
    """The same split contraction with the weight read in its forward layout
    (contraction index strided) and an E5 gradient operand."""
    g = I.normal_bf16(T, N, 1e-3, 37, 1, "cuda")
    w = I.normal_bf16(N, K, 0.02, 37, 2, "cuda")
    qg, qw = Quantised(ctx, g, O.E5, O.CONV_PAPER), Quantised(ctx, w, O.E4, O.CONV_PAPER)
    ref = O.linear_dgrad(qg.ref, qg.shift, qw.ref, qw.shift)
    dx = torch.full((T, K), float("nan"), dtype=torch.float32, device="cuda")
    ctx.linear_dgrad(qg.y, qg.bias, qw.y, None, qw.bias, dx)
    assert_gemm_close(dx.cpu().numpy(), ref)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


class _PtqLayer:
    """One weight tensor of config 4 quantised once on the GPU (fp8_ptq_weights) and once by the oracle; bytes,
    amax and bias compared in full here, then shared by every token count."""

    def __init__(self, ctx, lib, layer):
        wl = I.WORKLOADS["c4_llama70b_ptq"]
        l = wl.layers[layer]
        self.K, self.N, self.name = l.K, l.N, l.name
        w = I.layer_tensors(wl, layer, device="cuda", tokens=16, want=("w",))["w"]
        self.w8 = torch.empty((l.N, l.K), dtype=torch.uint8, device="cuda")
        self.amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        ctx.ptq_weights(w, lib.CONV_PAPER, self.w8, None, self.bias, self.amax)
        a, b, ref = O.quantise(bits_of(w), O.E4)
        del w
        assert float(self.amax.item()) == a and int(self.bias.item()) == b
        assert_codes_equal(u8(self.w8), ref, O.N_E4)
        self.ref, self.shift = ref, b + 1


_ptq_cache = {}


def _ptq_layer(ctx, lib, layer):
    if layer not in _ptq_cache:
        _ptq_cache.clear()            # one layer's bytes at a time (the largest holds 470 MB on each side)
        _ptq_cache[layer] = _PtqLayer(ctx, lib, layer)
    return _ptq_cache[layer]


@pytest.mark.parametrize("layer,tokens", [(l, t) for l in (0, 1, 2, 3) for t in (1, 16, 64, 2048)])
def test_llama70b_ptq_inference_layers(ctx, lib, layer, tokens):
    """Config 4: weights quantised once (post-training quantisation, Section 3.1), forward only; every layer at
    every token count of the config (decode 1 / 16 / 64, prefill 2048).  Weight bytes are checked in full, the
    activation's bytes in full, the output at 64 positions per 128 x 128 block, on eight whole blocks and on its
    first / last rows and columns."""
    wl = I.WORKLOADS["c4_llama70b_ptq"]
    pw = _ptq_layer(ctx, lib, layer)
    x = I.layer_tensors(wl, layer, device="cuda", tokens=tokens, want=("x",))["x"]
    qx = Quantised(ctx, x, O.E4, O.CONV_PAPER, transposed=False)
    y = torch.empty((tokens, pw.N), dtype=torch.bfloat16, device="cuda")
    ctx.linear_fwd(qx.y, qx.bias, pw.w8, pw.bias, y)
    y_inf = torch.empty_like(y)
    ctx.linear_infer(qx.y, qx.bias, pw.w8, pw.bias, y_inf)     # what the benchmark's forward-only workloads call
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    assert torch.equal(y.view(torch.int16), y_inf.view(torch.int16))
    if tokens <= 128:   # the benchmark's decode step: activation quantised by the matmul's own call
        x8, amax, bias, y_q, _ = _infer_cast(ctx, x, pw.w8, pw.bias, torch.bfloat16)
        assert float(amax.item()) == float(qx.amax.item()) and int(bias.item()) == qx.ref_bias
        assert_codes_equal(u8(x8), qx.ref, O.N_E4)
        assert torch.equal(y.view(torch.int16), y_q.view(torch.int16))
        assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    rng = np.random.default_rng(layer * 100 + tokens)
    rows, cols = tile_sample_positions(rng, tokens, pw.N)
    ref = O.linear_samples(O.FWD, qx.ref, O.N_E4, qx.shift, pw.ref, O.N_E4, pw.shift, rows, cols)
    frac = assert_bf16_within_one_ulp(bits_of(y)[rows, cols], ref)
    print(f"[parity] c4/{pw.name} T={tokens}: {rows.size} positions, {frac:.5f} through the cancellation branch")


def test_ptq_cache_is_released():
    _ptq_cache.clear()


def test_fused_epilogue_argument_errors(ctx, lib):
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    x8 = torch.zeros((32, 64), dtype=torch.uint8, device="cuda")
    w8 = torch.zeros((48, 64), dtype=torch.uint8, device="cuda")
    y = torch.zeros((32, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_act(x8, b, w8, b, None, None)                       # the activated output is mandatory
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_act(x8, b, w8, b, None, y, act=7)                   # unknown activation
    assert e.value.status == lib.ERR_DTYPE
    w8_odd = torch.zeros((44, 64), dtype=torch.uint8, device="cuda")       # N = 44: rows of y not 16-byte multiples
    y_odd = torch.zeros((32, 44), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_fwd_act(x8, b, w8_odd, b, None, y_odd)
    assert e.value.status == lib.ERR_ALIGN
    g8 = torch.zeros((32, 48), dtype=torch.uint8, device="cuda")
    dxa = torch.zeros((32, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_dgrad_act(g8, b, w8, None, b, None, None, dxa)          # no pre-activation given
    assert e.value.status == lib.ERR_NULL
    # a valid tiny call still works after the rejected ones
    ctx.linear_fwd_act(x8, b, w8, b, None, y)
    assert bool((y == 0).all()) and ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


@pytest.mark.parametrize("T", [16, 512])
def test_a_layer_replayed_from_a_cuda_graph_matches_the_eager_run(ctx, lib, T):
    """Quantise X (amax + bias + cast), forward matmul with output amax, for a decode-size batch (single launch
    cast, split contraction, finalize and matmul launched as programmatic dependents) and a training-size one:
    captured once, replayed on fresh inputs, the results must equal the eager calls' bit for bit."""
    K, N = 2048, 1536
    w = I.normal_bf16(N, K, 0.02, 55, 2, "cuda")
    qw = Quantised(ctx, w, O.E4, O.CONV_PAPER)
    x = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    x8 = torch.empty((T, K), dtype=torch.uint8, device="cuda")
    ax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bx = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ay = torch.zeros(1, dtype=torch.float32, device="cuda")

    def layer():
        ctx.cast_e4(x, None, d_amax_out=ax, d_bias_out=bx, y=x8)
        ctx.linear_fwd(x8, bx, qw.y, qw.bias, y, d_amax_y=ay)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        x.copy_(I.normal_bf16(T, K, 1.0, 56, 1, "cuda"))
        layer()
        with torch.cuda.graph(g, stream=side):
            layer()
    torch.cuda.current_stream().wait_stream(side)
    for seed, scale in ((57, 1.0), (58, 300.0), (59, 0.004)):
        x.copy_(I.normal_bf16(T, K, scale, seed, 1, "cuda"))
        g.replay()
        torch.cuda.synchronize()
        got = (y.clone(), x8.clone(), float(ax.item()), int(bx.item()), float(ay.item()))
        y.zero_(); x8.zero_(); ax.zero_(); bx.zero_(); ay.zero_()
        layer()
        torch.cuda.synchronize()
        assert torch.equal(got[0], y) and torch.equal(got[1], x8)
        assert got[2:] == (float(ax.item()), int(bx.item()), float(ay.item()))
        assert got[3] == O.scaling_bias(O.amax(bits_of(x)), O.E4)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
