"""fp8_cast_predicted: FP8-AMAX in one pass when the bias guess holds.  Whatever
the guess, amax, bias and bytes must equal the oracle's (and therefore the
two-launch path's), and the hit / miss counters must tell the two cases apart."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_codes_equal, bits_of, u8

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


def _host(t):
    return bits_of(t) if t.dtype == torch.bfloat16 else t.detach().contiguous().cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
@pytest.mark.parametrize("kind", [O.E4, O.E5])
@pytest.mark.parametrize("shape", [(1, 5), (64, 64), (300, 520), (1024, 4096)])
def test_any_guess_gives_the_exact_result(ctx, lib, dtype, kind, shape):
    g = torch.Generator(device="cuda").manual_seed(shape[0] + 17 * kind)
    x = (torch.randn(shape, generator=g, device="cuda") * 0.02).to(dtype)
    a, b, want = O.quantise(_host(x), kind, O.CONV_PAPER, 0)
    fmt = O.native_format(kind)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(shape, dtype=torch.uint8, device="cuda")
    ctx.prediction_stats(clear=True)
    ctx.device_flags(clear=True)
    guesses = [b, b + 1, b - 7, 0, 2 ** 31 - 1, -2 ** 31, b]
    expected_hits = sum(1 for q in guesses if q == b)
    for guess in guesses:
        bias.fill_(guess)
        y.fill_(0x55)
        amax.fill_(-1.0)
        ctx.cast_predicted(kind, x, amax, bias, y)
        assert float(amax.item()) == a and int(bias.item()) == b, guess
        assert_codes_equal(u8(y), want, fmt)
    hits, misses = ctx.prediction_stats(clear=True)
    assert (hits, misses) == (expected_hits, len(guesses) - expected_hits)
    assert ctx.prediction_stats() == (0, 0)


def test_steady_state_and_a_moving_tensor(ctx, lib):
    """Same tensor every step: one miss, then hits.  A tensor whose scale doubles every step: all misses, and
    still the exact result every time."""
    x = torch.randn((512, 1024), device="cuda").to(torch.bfloat16)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    y = torch.empty((512, 1024), dtype=torch.uint8, device="cuda")
    ctx.prediction_stats(clear=True)
    for _ in range(6):
        ctx.cast_predicted(lib.E4, x, amax, bias, y)
    assert ctx.prediction_stats(clear=True) == (5, 1)
    for k in range(5):
        xk = (x.float() * 2.0 ** (k + 1)).to(torch.bfloat16)
        a, b, want = O.quantise(bits_of(xk), O.E4)
        ctx.cast_predicted(lib.E4, xk, amax, bias, y)
        assert int(bias.item()) == b
        assert_codes_equal(u8(y), want, O.N_E4)
    assert ctx.prediction_stats(clear=True) == (0, 5)


def test_saturation_flag_only_reports_the_true_bias(ctx, lib):
    ctx.device_flags(clear=True)
    x = torch.full((256, 256), 3.0, dtype=torch.bfloat16, device="cuda")   # 3 * 2^7 = 384 fits natively: no clipping
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.full((1,), 20, dtype=torch.int32, device="cuda")          # wildly too large a guess: pass one clips
    y = torch.empty((256, 256), dtype=torch.uint8, device="cuda")
    ctx.cast_predicted(lib.E4, x, amax, bias, y)
    assert int(bias.item()) == 6 and ctx.device_flags() == 0
    assert_codes_equal(u8(y), O.cast(bits_of(x), 7, O.N_E4), O.N_E4)


def test_strided_input_takes_the_two_launch_path(ctx, lib):
    big = torch.randn((128, 300), device="cuda").to(torch.bfloat16)
    view = big[:, 8:264]
    a, b, want = O.quantise(bits_of(view), O.E4)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty((128, 256), dtype=torch.uint8, device="cuda")
    ctx.cast_predicted(lib.E4, view, amax, bias, y, rows=128, cols=256, ld=300)
    assert float(amax.item()) == a and int(bias.item()) == b
    assert_codes_equal(u8(y), want, O.N_E4)


@pytest.mark.parametrize("shape,transposed", [((512, 1024), False), ((300, 520), False), ((256, 384), True)])
def test_delayed_scaling_casts_with_the_given_bias_and_reports_the_next_one(ctx, lib, shape, transposed):
    """fp8_cast_e4 with a bias AND output slots: bytes follow the given bias; amax and the bias Eq. 3 gives for
    this tensor come out of the same call for the next step."""
    x = (torch.randn(shape, device="cuda") * 0.05).to(torch.bfloat16)
    xb = bits_of(x)
    a, b_true = O.amax(xb), None
    b_true = O.scaling_bias(a, O.E4)
    stale = b_true - 2                      # e.g. last step's tensor was four times larger
    bias_in = torch.full((1,), stale, dtype=torch.int32, device="cuda")
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias_next = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(shape, dtype=torch.uint8, device="cuda")
    y_t = torch.empty(shape[::-1], dtype=torch.uint8, device="cuda") if transposed else None
    ctx.cast_e4(x, bias_in, d_amax_out=amax, d_bias_out=bias_next, y=y, y_t=y_t)
    assert_codes_equal(u8(y), O.cast(xb, stale + 1, O.N_E4), O.N_E4)
    if transposed:
        assert_codes_equal(u8(y_t), O.cast(xb, stale + 1, O.N_E4).T, O.N_E4)
    assert float(amax.item()) == a and int(bias_next.item()) == b_true and int(bias_in.item()) == stale
    # in place: the same word holds the bias used and then the next one
    ctx.cast_e4(x, bias_in, d_amax_out=amax, d_bias_out=bias_in, y=y, y_t=y_t)
    assert_codes_equal(u8(y), O.cast(xb, stale + 1, O.N_E4), O.N_E4)
    assert int(bias_in.item()) == b_true


def test_config2_gradient_magnitude_moves_every_step(ctx, lib):
    """Config 2: the output gradient of the QKV layer is redrawn every step with a log-uniform magnitude in
    2^-12 .. 2^-4, so its E5 bias has to move.  At each of 16 steps amax and bias must equal the oracle's, the
    bytes must match on sampled rows, both through the two-launch path and through the one-pass path (which
    mostly mispredicts here and must still be exact)."""
    from paper_2309_17224_b200 import inputs as I
    wl = I.WORKLOADS["c2_gpt"]
    T, N = wl.tokens, wl.layers[0].N
    amax = torch.zeros(2, dtype=torch.float32, device="cuda")
    bias = torch.zeros(2, dtype=torch.int32, device="cuda")
    y = torch.empty((T, N), dtype=torch.uint8, device="cuda")
    y2 = torch.empty((T, N), dtype=torch.uint8, device="cuda")
    rng = np.random.default_rng(2)
    seen = set()
    ctx.prediction_stats(clear=True)
    for step in range(16):
        g = I.layer_tensors(wl, 0, device="cuda", step=step, want=("g",))["g"]
        gb = bits_of(g)
        a = O.amax(gb)
        b = O.scaling_bias(a, O.E5)
        seen.add(b)
        ctx.cast_e5(g, None, d_amax_out=amax[0:1], d_bias_out=bias[0:1], y=y)
        ctx.cast_predicted(lib.E5, g, amax[1:2], bias[1:2], y2)
        assert amax.tolist() == [a, a] and bias.tolist() == [b, b], step
        rows = np.sort(rng.choice(T, size=64, replace=False))
        want = O.cast(gb[rows], b, O.N_E5)
        assert_codes_equal(u8(y)[rows], want, O.N_E5)
        assert torch.equal(y, y2)
    hits, misses = ctx.prediction_stats(clear=True)
    assert hits + misses == 16 and misses >= 8
    assert len(seen) >= 5 and max(seen) - min(seen) >= 4
