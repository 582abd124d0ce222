"""GPU parity: amax, scaling bias and scale-and-cast against the CPU oracle,
bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_codes_equal, bf16_from_bits, bits_of, u8

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


def _dev_scalar(dtype, value=0):
    return torch.full((1,), value, dtype=dtype, device="cuda")


def _same_float(a: float, b: float) -> bool:
    return (np.isnan(a) and np.isnan(b)) or a == b


def _gpu_amax(ctx, x, **kw):
    out = _dev_scalar(torch.float32, -1.0)
    ctx.amax(x, out, **kw)
    return float(out.item())


@pytest.mark.parametrize("shape", [(1, 1), (1, 7), (3, 8), (256, 768), (300, 520), (129, 257), (1024, 4096), (5, 100003)])
def test_amax_contiguous(ctx, shape):
    g = torch.Generator(device="cuda").manual_seed(shape[0] * 7919 + shape[1])
    x = (torch.randn(shape, generator=g, device="cuda") * 3.0).to(torch.bfloat16)
    assert _gpu_amax(ctx, x) == O.amax(bits_of(x))
    # the maximum sitting at the very last / very first element, negative
    x[-1, -1] = -4096.0
    assert _gpu_amax(ctx, x) == 4096.0
    x[0, 0] = 8192.0
    assert _gpu_amax(ctx, x) == 8192.0


def test_amax_strided_and_unaligned(ctx):
    g = torch.Generator(device="cuda").manual_seed(5)
    big = torch.randn((70, 264), generator=g, device="cuda").to(torch.bfloat16)
    big[:, 200:] = 1000.0  # outside every view below
    for cols, off in ((200, 0), (192, 0), (199, 1), (64, 3)):
        view = big[:, off:off + cols]
        want = O.amax(bits_of(view))
        assert _gpu_amax(ctx, view, rows=70, cols=cols, ld=264) == want


def test_amax_special_values(ctx):
    x = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    assert _gpu_amax(ctx, x) == 0.0
    x[3, 3] = -0.0
    assert _gpu_amax(ctx, x) == 0.0
    sub = bf16_from_bits(np.array([[0x8001, 0x0000]], dtype=np.uint16), "cuda")
    assert _gpu_amax(ctx, sub) == 2.0 ** -133
    x[10, 10] = float("inf")
    assert _gpu_amax(ctx, x) == float("inf")
    x[20, 20] = float("nan")
    assert np.isnan(_gpu_amax(ctx, x)) and np.isnan(O.amax(bits_of(x)))
    # repeated calls reuse the reduction slots: the result must not depend on history
    y = torch.ones((128, 128), dtype=torch.bfloat16, device="cuda")
    for _ in range(200):
        assert _gpu_amax(ctx, y) == 1.0


def test_scaling_bias_kernel_matches_oracle(ctx, lib):
    vals = [0.0, 1e-45, 2.0 ** -133, 1e-30, 0.005, 0.08, 1.0, 1.875, 1.8828125, 5.0, 120.0, 240.0, 241.0, 448.0,
            449.0, 57344.0, 57600.0, 3.0e38, float("inf"), float("nan")]
    amax = _dev_scalar(torch.float32)
    bias = _dev_scalar(torch.int32, 12345)
    for v in vals:
        for fmt, conv in ((lib.E4, lib.CONV_PAPER), (lib.E4, lib.CONV_NATIVE), (lib.E5, lib.CONV_PAPER)):
            for margin in (0, 3):
                amax.fill_(v)
                ctx.scaling_bias(amax, fmt, conv, margin, bias)
                assert int(bias.item()) == O.scaling_bias(v, fmt, conv, margin), (v, fmt, conv, margin)
    flags = ctx.device_flags(clear=True)
    assert flags & lib.FLAG_ZERO_AMAX and flags & lib.FLAG_NONFINITE_AMAX
    assert ctx.device_flags() == 0


def _all_bf16(device="cuda"):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(256, 256)
    return bits, bf16_from_bits(bits, device)


@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_cast_every_bf16_value_at_every_shift(ctx, lib, kind):
    """All 65 536 input bit patterns x every shift a bias can produce."""
    bits, x = _all_bf16()
    fmt = O.native_format(kind)
    cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
    bias = _dev_scalar(torch.int32)
    y = torch.empty((256, 256), dtype=torch.uint8, device="cuda")
    y_t = torch.empty((256, 256), dtype=torch.uint8, device="cuda")
    for b in range(-151, 152):
        conv = lib.CONV_PAPER if b % 2 else lib.CONV_NATIVE
        bias.fill_(b)
        want = O.cast(bits, b + O.delta(kind, conv), fmt)
        if b % 3 == 0:  # flat kernel
            cast(x, bias, conv=conv, y=y)
            assert_codes_equal(u8(y), want, fmt)
        else:           # tiled kernel, both layouts
            cast(x, bias, conv=conv, y=y, y_t=y_t)
            assert_codes_equal(u8(y), want, fmt)
            assert_codes_equal(u8(y_t), want.T, fmt)


@pytest.mark.parametrize("shape", [(1, 1), (1, 7), (4, 16), (128, 128), (129, 257), (300, 520), (256, 768), (257, 131), (640, 1024)])
@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_cast_shapes_with_and_without_transpose(ctx, lib, kind, shape):
    g = torch.Generator(device="cuda").manual_seed(shape[0] * 31 + shape[1])
    x = (torch.randn(shape, generator=g, device="cuda") * 0.7).to(torch.bfloat16)
    x[0, 0] = float("nan") if shape[1] > 1 else 1.0
    xb = bits_of(x)
    fmt = O.native_format(kind)
    cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
    a = O.amax(bits_of(torch.nan_to_num(x, nan=0.0)))
    b = O.scaling_bias(a, kind)
    want = O.cast(xb, b + O.delta(kind, O.CONV_PAPER), fmt)
    bias = _dev_scalar(torch.int32, b)
    rows, cols = shape
    y = torch.full((rows * cols + 64,), 0xAB, dtype=torch.uint8, device="cuda")
    y_t = torch.full((rows * cols + 64,), 0xCD, dtype=torch.uint8, device="cuda")
    for use_y, use_t in ((True, False), (False, True), (True, True)):
        y.fill_(0xAB)
        y_t.fill_(0xCD)
        cast(x, bias, y=y if use_y else None, y_t=y_t if use_t else None)
        if use_y:
            assert_codes_equal(u8(y[:rows * cols]).reshape(rows, cols), want, fmt)
        if use_t:
            assert_codes_equal(u8(y_t[:rows * cols]).reshape(cols, rows), want.T, fmt)
        # nothing written past the end of either output
        assert bool((y[rows * cols:] == 0xAB).all()) and bool((y_t[rows * cols:] == 0xCD).all())


def test_cast_strided_input(ctx, lib):
    g = torch.Generator(device="cuda").manual_seed(17)
    big = torch.randn((200, 400), generator=g, device="cuda").to(torch.bfloat16)
    bias = _dev_scalar(torch.int32, 4)
    for cols, off in ((256, 0), (250, 8), (129, 1)):
        view = big[:, off:off + cols]
        want = O.cast(bits_of(view), 5, O.N_E4)
        y = torch.empty((200, cols), dtype=torch.uint8, device="cuda")
        y_t = torch.empty((cols, 200), dtype=torch.uint8, device="cuda")
        ctx.cast_e4(view, bias, y=y, y_t=y_t, rows=200, cols=cols, ld=400)
        assert_codes_equal(u8(y), want, O.N_E4)
        assert_codes_equal(u8(y_t), want.T, O.N_E4)


@pytest.mark.parametrize("kind,conv,margin", [(O.E4, O.CONV_PAPER, 0), (O.E4, O.CONV_NATIVE, 0), (O.E5, O.CONV_PAPER, 0),
                                              (O.E5, O.CONV_PAPER, 3)])
@pytest.mark.parametrize("std", [1e-5, 0.02, 1.0, 4000.0])
def test_fused_amax_bias_cast(ctx, lib, kind, conv, margin, std):
    """FP8-AMAX in one call: amax, bias and bytes all equal the oracle's."""
    g = torch.Generator(device="cuda").manual_seed(int(std * 1e6) % 9973 + kind)
    x = (torch.randn((384, 640), generator=g, device="cuda") * std).to(torch.bfloat16)
    a, b, want, want_t = O.quantise(bits_of(x), kind, conv, margin, transposed=True)
    amax = _dev_scalar(torch.float32, -1.0)
    bias = _dev_scalar(torch.int32, 777)
    y = torch.empty((384, 640), dtype=torch.uint8, device="cuda")
    y_t = torch.empty((640, 384), dtype=torch.uint8, device="cuda")
    cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
    cast(x, None, conv=conv, margin=margin, d_amax_out=amax, d_bias_out=bias, y=y, y_t=y_t)
    assert float(amax.item()) == a and int(bias.item()) == b
    assert_codes_equal(u8(y), want, O.native_format(kind))
    assert_codes_equal(u8(y_t), want_t, O.native_format(kind))
    y.zero_()
    cast(x, None, conv=conv, margin=margin, d_amax_out=amax, d_bias_out=bias, y=y)
    assert_codes_equal(u8(y), want, O.native_format(kind))


def test_ptq_weights_equals_separate_steps(ctx, lib):
    g = torch.Generator(device="cuda").manual_seed(23)
    w = (torch.randn((768, 512), generator=g, device="cuda") * 0.015).to(torch.bfloat16)
    a, b, want, want_t = O.quantise(bits_of(w), O.E4, O.CONV_PAPER, 0, transposed=True)
    w8 = torch.empty((768, 512), dtype=torch.uint8, device="cuda")
    w8_t = torch.empty((512, 768), dtype=torch.uint8, device="cuda")
    amax = _dev_scalar(torch.float32)
    bias = _dev_scalar(torch.int32)
    ctx.ptq_weights(w, lib.CONV_PAPER, w8, w8_t, bias, amax)
    assert float(amax.item()) == a and int(bias.item()) == b
    assert_codes_equal(u8(w8), want, O.N_E4)
    assert_codes_equal(u8(w8_t), want_t, O.N_E4)
    # the same through the separate entry points
    amax2, bias2 = _dev_scalar(torch.float32), _dev_scalar(torch.int32)
    w8b = torch.empty_like(w8)
    ctx.amax(w, amax2)
    ctx.scaling_bias(amax2, lib.E4, lib.CONV_PAPER, 0, bias2)
    ctx.cast_e4(w, bias2, y=w8b)
    assert torch.equal(w8, w8b) and int(bias2.item()) == b


def test_saturation_flag_and_constant_scale(ctx, lib):
    """A caller-chosen constant bias (FP8-CSCALE) that is too large clips and
    raises the sticky flag; a safe one does not."""
    ctx.device_flags(clear=True)
    x = torch.full((64, 64), 3.0, dtype=torch.bfloat16, device="cuda")
    y = torch.empty((64, 64), dtype=torch.uint8, device="cuda")
    bias = _dev_scalar(torch.int32, 2)
    ctx.cast_e4(x, bias, y=y)
    assert ctx.device_flags() == 0
    assert_codes_equal(u8(y), O.cast(bits_of(x), 3, O.N_E4), O.N_E4)
    bias.fill_(9)  # 3 * 2^10 = 3072 > 448
    ctx.cast_e4(x, bias, y=y)
    assert ctx.device_flags() & lib.FLAG_SATURATED
    assert bool((y == 0x7E).all())


@pytest.mark.parametrize("top,flag", [(240.0, True), (236.0, True), (233.0, True), (232.0, False), (200.0, False)])
def test_paper_convention_raises_saturated_when_amax_rounds_to_the_240_code(ctx, lib, top, flag):
    """Just-in-time FP8-AMAX under the paper convention: a scaled amax in (232, 240] would take the paper format's
    top code, which has no native byte; the cast emits 224 (byte 0x7E) and raises FP8_FLAG_SATURATED.  Same bytes
    as the oracle; the native convention raises nothing."""
    x = (torch.randn((64, 256), device="cuda") * 20.0).clamp(-200, 200).to(torch.bfloat16)
    x[3, 5], x[60, 255] = top, -top
    for conv, expect in ((lib.CONV_PAPER, flag), (lib.CONV_NATIVE, False)):
        ctx.device_flags(clear=True)
        y = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        amax, bias = _dev_scalar(torch.float32), _dev_scalar(torch.int32, 99)
        ctx.cast_e4(x, None, conv=conv, d_amax_out=amax, d_bias_out=bias, y=y)
        a, b, ref = O.quantise(bits_of(x), O.E4, conv)
        assert (float(amax.item()), int(bias.item())) == (a, b) and a == top and (b == 0 or conv == lib.CONV_NATIVE)
        assert_codes_equal(u8(y), ref, O.N_E4)
        assert bool(ctx.device_flags(clear=True) & lib.FLAG_SATURATED) == expect
        if conv == lib.CONV_PAPER and top > 216:
            assert u8(y)[3, 5] == 0x7E and u8(y)[60, 255] == 0xFE


def test_argument_errors(ctx, lib):
    x = torch.zeros((16, 16), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((16, 16), dtype=torch.uint8, device="cuda")
    bias = _dev_scalar(torch.int32)
    with pytest.raises(lib.Fp8Error) as e:
        ctx.cast_e4(x, bias, y=None, y_t=None)
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.cast_e4(x, None, y=y)  # FP8-AMAX needs somewhere to put amax and bias
    assert e.value.status == lib.ERR_NULL
    with pytest.raises(lib.Fp8Error) as e:
        ctx.cast_e4(x, bias, y=y, rows=16, cols=16, ld=8)
    assert e.value.status == lib.ERR_SHAPE
    raw = lib.raw()
    assert raw.fp8_amax(ctx._h, x.data_ptr(), 7, 16, 16, 16, bias.data_ptr(), None) == lib.ERR_DTYPE


# ----------------------------------------------------------------------------
# fp16 and fp32 inputs (the paper's own tensors are FP16)
# ----------------------------------------------------------------------------

def _host(t):
    """torch fp16 / fp32 tensor -> numpy array the oracle accepts."""
    return t.detach().contiguous().cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float16, torch.float32])
@pytest.mark.parametrize("shape", [(1, 1), (1, 5), (3, 8), (256, 768), (300, 520), (129, 257), (5, 100003)])
def test_amax_fp16_fp32(ctx, dtype, shape):
    g = torch.Generator(device="cuda").manual_seed(shape[0] * 131 + shape[1])
    x = (torch.randn(shape, generator=g, device="cuda") * 3.0).to(dtype)
    assert _gpu_amax(ctx, x) == O.amax(_host(x))
    x[-1, -1] = -4096.0
    assert _gpu_amax(ctx, x) == 4096.0
    if shape[1] >= 8:
        big = torch.zeros((shape[0], shape[1] + 24), dtype=dtype, device="cuda")
        big[:, 5:5 + shape[1]] = x
        big[:, :5] = 30000.0
        view = big[:, 5:5 + shape[1]]
        assert _gpu_amax(ctx, view, rows=shape[0], cols=shape[1], ld=shape[1] + 24) == O.amax(_host(view))
    x[0, 0] = float("inf")
    assert _gpu_amax(ctx, x) == float("inf")
    x[0, 0] = float("nan")
    assert np.isnan(_gpu_amax(ctx, x))


@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_cast_every_fp16_value(ctx, lib, kind):
    """All 65 536 fp16 bit patterns at every shift that can bring one of them into the FP8 range."""
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16).view(np.float16).reshape(256, 256)
    x = torch.from_numpy(h.copy()).cuda()
    fmt = O.native_format(kind)
    cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
    bias = _dev_scalar(torch.int32)
    y = torch.empty((256, 256), dtype=torch.uint8, device="cuda")
    y_t = torch.empty((256, 256), dtype=torch.uint8, device="cuda")
    for b in list(range(-36, 44)) + [-150, -127, 126, 140]:
        bias.fill_(b)
        want = O.cast(h, b + O.delta(kind, O.CONV_PAPER), fmt)
        if b % 2:
            cast(x, bias, y=y)
        else:
            cast(x, bias, y=y, y_t=y_t)
            assert_codes_equal(u8(y_t), want.T, fmt)
        assert_codes_equal(u8(y), want, fmt)


@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_cast_fp32_values_and_extremes(ctx, lib, kind):
    rng = np.random.default_rng(kind + 10)
    bits = rng.integers(0, 2 ** 32, size=(384, 512), dtype=np.uint64).astype(np.uint32)   # every exponent, both signs, NaNs too
    bits[0, :8] = [0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0x7F800000, 0xFF800000, 0x7FC00000, 0x80000000]
    f = bits.view(np.float32)
    x = torch.from_numpy(f.copy()).cuda()
    fmt = O.native_format(kind)
    cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
    bias = _dev_scalar(torch.int32)
    y = torch.empty(f.shape, dtype=torch.uint8, device="cuda")
    y_t = torch.empty(f.shape[::-1], dtype=torch.uint8, device="cuda")
    for b in (-150, -130, -126, -60, -7, 0, 3, 40, 100, 127, 140, 152):
        bias.fill_(b)
        want = O.cast(f, b + O.delta(kind, O.CONV_PAPER), fmt)
        cast(x, bias, y=y, y_t=y_t)
        assert_codes_equal(u8(y), want, fmt)
        assert_codes_equal(u8(y_t), want.T, fmt)
        cast(x, bias, y=y)
        assert_codes_equal(u8(y), want, fmt)


@pytest.mark.parametrize("dtype", [torch.float16, torch.float32])
@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_fused_amax_bias_cast_fp16_fp32(ctx, lib, dtype, kind):
    g = torch.Generator(device="cuda").manual_seed(77 + kind)
    for shape, std in (((384, 640), 0.02), ((129, 257), 3.0), ((64, 4096), 1e-3)):
        x = (torch.randn(shape, generator=g, device="cuda") * std).to(dtype)
        a, b, want, want_t = O.quantise(_host(x), kind, O.CONV_PAPER, 0, transposed=True)
        amax = _dev_scalar(torch.float32, -1.0)
        bias = _dev_scalar(torch.int32, 777)
        y = torch.empty(shape, dtype=torch.uint8, device="cuda")
        y_t = torch.empty(shape[::-1], dtype=torch.uint8, device="cuda")
        cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
        cast(x, None, d_amax_out=amax, d_bias_out=bias, y=y, y_t=y_t)
        assert float(amax.item()) == a and int(bias.item()) == b
        assert_codes_equal(u8(y), want, O.native_format(kind))
        assert_codes_equal(u8(y_t), want_t, O.native_format(kind))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
@pytest.mark.parametrize("shape", [(1, 5), (1, 8192), (16, 8192), (64, 8192), (129, 257), (3, 8), (512, 1024), (1024, 1024)])
def test_fp8_amax_on_small_tensors_single_launch(ctx, lib, dtype, shape):
    """Decode-size activations: the whole tensor is quantised by one cluster in one launch (row-major output,
    FP8-AMAX); larger ones fall through to the two-launch path.  Same results either way."""
    g = torch.Generator(device="cuda").manual_seed(shape[0] * 7 + shape[1])
    for kind, std in ((O.E4, 1.0), (O.E5, 1e-4)):
        x = (torch.randn(shape, generator=g, device="cuda") * std).to(dtype)
        if shape[1] >= 8:
            x[0, 3] = 100.0 * std   # an outlier decides the bias
        host = bits_of(x) if dtype == torch.bfloat16 else _host(x)
        a, b, want = O.quantise(host, kind, O.CONV_PAPER, 0)
        amax = _dev_scalar(torch.float32, -1.0)
        bias = _dev_scalar(torch.int32, 777)
        y = torch.full((shape[0] * shape[1] + 32,), 0xEE, dtype=torch.uint8, device="cuda")
        cast = ctx.cast_e4 if kind == O.E4 else ctx.cast_e5
        cast(x, None, d_amax_out=amax, d_bias_out=bias, y=y)
        assert float(amax.item()) == a and int(bias.item()) == b
        n = shape[0] * shape[1]
        assert_codes_equal(u8(y[:n]).reshape(shape), want, O.native_format(kind))
        assert bool((y[n:] == 0xEE).all())
    z = torch.zeros(shape, dtype=dtype, device="cuda")
    ctx.device_flags(clear=True)
    ctx.cast_e4(z, None, d_amax_out=amax, d_bias_out=bias, y=y)
    assert float(amax.item()) == 0.0 and int(bias.item()) == 0 and ctx.device_flags() & lib.FLAG_ZERO_AMAX


@pytest.mark.parametrize("kind", [O.E4, O.E5])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_range_statistics_of_a_constant_bias_sweep(ctx, lib, kind, dtype):
    """FP8-CSCALE style sweep: for each candidate bias the counts of clipped / flushed / subnormal elements must
    equal what the oracle's bytes say."""
    g = torch.Generator(device="cuda").manual_seed(5 + kind)
    x = (torch.randn((257, 383), generator=g, device="cuda") * 0.3).to(dtype)
    x[0, :6] = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 1e-30], device="cuda").to(dtype)
    host = bits_of(x) if dtype == torch.bfloat16 else _host(x)
    xv = x.double().cpu().numpy()
    fmt = O.native_format(kind)
    m_bits = 3 if kind == O.E4 else 2
    bias = _dev_scalar(torch.int32)
    counts = torch.full((4,), 99, dtype=torch.int64, device="cuda")
    results = {}
    for b in (-12, -4, 0, 3, 8, 15, 24):
        bias.fill_(b)
        ctx.range_stats(kind, x, bias, counts)
        s = b + O.delta(kind, O.CONV_PAPER)
        codes = O.cast(host, s, fmt) & 0x7F
        v = np.abs(np.ldexp(xv, s))
        notnan = ~np.isnan(xv)
        nz = notnan & np.isfinite(xv) & (xv != 0)
        clipped = notnan & ((v > 464.0) if kind == O.E4 else (v >= 61440.0))
        want = [int(clipped.sum()), int((nz & (codes == 0)).sum()),
                int((notnan & (codes > 0) & (codes < (1 << m_bits))).sum()), int(nz.sum())]
        assert counts.tolist() == want, (b, counts.tolist(), want)
        results[b] = want
    # the sweep shows the window: small biases flush, large ones clip
    assert results[-12][1] > results[3][1] and results[24][0] > results[3][0]


@pytest.mark.parametrize("length", [1, 4, 33, 100])
@pytest.mark.parametrize("kind", [O.E4, O.E5])
def test_amax_history_ring(ctx, lib, length, kind):
    """fp8_amax_history_bias keeps the last `length` amax values of a tensor in a ring and returns Eq. 3 on the
    largest of them minus the margin; checked against the oracle's rule on the same window after every push,
    through several wraps of the ring."""
    rng = np.random.default_rng(length * 10 + kind)
    hist = torch.zeros(length, dtype=torch.float32, device="cuda")
    cursor = torch.zeros(1, dtype=torch.int32, device="cuda")
    new = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.zeros(1, dtype=torch.int32, device="cuda")
    margin = 2
    pushed = []
    for step in range(3 * length + 5):
        a = float(np.float32(2.0 ** rng.uniform(-30, 30)))
        pushed.append(a)
        new.fill_(a)
        ctx.amax_history_bias(hist, cursor, new, kind, bias, margin=margin)
        window = pushed[-length:]
        assert int(bias.item()) == O.history_bias(window, kind, O.CONV_PAPER, margin), step
        assert int(cursor.item()) == (step + 1) % length
    assert sorted(hist.cpu().tolist()) == sorted(pushed[-length:])
    assert ctx.device_flags(clear=True) == 0
    # nothing but zeros in the window: bias 0 and the zero-amax flag, as for fp8_scaling_bias
    hist.zero_()
    new.zero_()
    ctx.amax_history_bias(hist, cursor, new, kind, bias)
    assert int(bias.item()) == 0 and ctx.device_flags(clear=True) & lib.FLAG_ZERO_AMAX
    with pytest.raises(lib.Fp8Error) as e:
        ctx.amax_history_bias(hist[:0], cursor, new, kind, bias)
    assert e.value.status in (lib.ERR_SHAPE, lib.ERR_NULL)


def test_bias_log_ring_wraps_and_mode_breaks_ties_downwards(ctx, lib):
    """fp8_bias_log_append on a ring of 10 records through several wraps, fp8_bias_mode on what the ring holds."""
    ring = torch.zeros((10, 4), dtype=torch.int32, device="cuda")
    head = torch.zeros(1, dtype=torch.int64, device="cuda")
    kept = []          # what a ring of 10 must hold
    biases = [[3, 7, -2], [3, 6, -2], [4, 6, -1], [4, 7, -1], [5, 7, -2], [3, 7, -2], [9, 9, 9]]
    for step, b in enumerate(biases):
        amax = torch.tensor([1.5 + step, 0.25, 100.0 * (step + 1)], dtype=torch.float32, device="cuda")
        ctx.bias_log_append(ring, head, step, 40, amax, torch.tensor(b, dtype=torch.int32, device="cuda"))
        kept += [(step, 40 + i, float(amax[i].item()), b[i]) for i in range(3)]
    n = len(kept)
    assert int(head.item()) == n
    host = ring.cpu()
    amax_f = host[:, 2].contiguous().view(torch.float32)
    for k in range(n - 10, n):
        r = host[k % 10]
        assert (int(r[0]), int(r[1]), float(amax_f[k % 10]), int(r[3])) == kept[k]
    mode, count, samples = (torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(3))
    live = kept[n - 10:]
    for tid in (40, 41, 42, 43):
        for lo, hi in ((0, 99), (4, 5), (6, 6), (50, 60)):
            ctx.bias_mode(ring, head, tid, lo, hi, mode, count, samples)
            seq = [b for (s_, t_, _, b) in live if t_ == tid and lo <= s_ <= hi]
            assert (int(mode.item()), int(count.item())) == O.bias_mode(seq) and int(samples.item()) == len(seq)
    # a tie: biases 4 and 6 twice each -> the smaller
    ring.zero_(); head.zero_()
    for step, b in enumerate((6, 4, 6, 4, 9)):
        ctx.bias_log_append(ring, head, step, 0, torch.ones(1, device="cuda"), torch.tensor([b], dtype=torch.int32, device="cuda"))
    ctx.bias_mode(ring, head, 0, 0, 10, mode, count)
    assert (int(mode.item()), int(count.item())) == (4, 2)
    with pytest.raises(lib.Fp8Error) as e:
        ctx.bias_log_append(ring, head, 0, 0, torch.ones(11, device="cuda"), torch.ones(11, dtype=torch.int32, device="cuda"))
    assert e.value.status == lib.ERR_SHAPE
