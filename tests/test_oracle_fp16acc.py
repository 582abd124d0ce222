"""Pins of the oracle's FP16-accumulation matmuls (Fig. 3b, Section 2.4, the margin of Section 3.2)."""
import numpy as np

import oracle as O


def _codes(fmt, values):
    return np.array([[O.encode(fmt, v) for v in row] for row in values], dtype=np.uint8)


def test_small_exact_sums_need_no_rounding():
    """Sums that are exactly representable in FP16 at every step equal the FP32-accumulate oracle's exact value."""
    rng = np.random.default_rng(0)
    x8 = _codes(O.N_E4, rng.integers(-4, 5, size=(5, 64)).astype(float))
    w8 = _codes(O.N_E4, rng.integers(-4, 5, size=(7, 64)).astype(float))
    for chunk in (1, 16, 64):
        got = O.linear_fwd_fp16acc(x8, 2, w8, 1, chunk=chunk)
        want = O.linear_fwd(x8, 2, w8, 1).f64
        assert np.array_equal(got.f64, want) and not got.overflowed.any()


def test_rounding_happens_once_per_chunk_and_follows_ieee_half():
    """2048 + 1 is not an FP16 number (spacing 2 above 2048): added one at a time the ones are lost (each tie goes to
    the even neighbour 2048); added as one exact chunk of 64 they survive.  The closed forms below are plain IEEE
    half arithmetic."""
    x8 = _codes(O.N_E4, [[256.0] + [1.0] * 64])          # one row: 256 then 64 ones
    w8 = _codes(O.N_E4, [[8.0] + [1.0] * 64])            # 256 * 8 = 2048, then 64 products of 1
    assert O.linear_fwd_fp16acc(x8, 0, w8, 0, chunk=1).f64[0, 0] == 2048.0
    assert O.linear_fwd_fp16acc(x8, 0, w8, 0, chunk=65).f64[0, 0] == 2112.0
    # chunk = 5: 2048 + 1 + 1 + 1 + 1 = 2052 exactly, then twelve chunks of five ones: 2057 is not representable
    # (spacing 2) and lies between 2056 and 2058; nearest even significand is 2056; ... computed with numpy's half
    acc = np.float16(0)
    terms = [2048.0] + [1.0] * 64
    for k0 in range(0, 65, 5):
        acc = np.float16(float(acc) + sum(terms[k0:k0 + 5]))
    assert O.linear_fwd_fp16acc(x8, 0, w8, 0, chunk=5).f64[0, 0] == float(acc)


def test_unscale_is_done_in_fp16():
    """Eq. 2 on an FP16 output: exact inside the normal range, one rounding into the subnormal range, zero below it,
    infinity above 65504."""
    x8, w8 = _codes(O.N_E4, [[3.0]]), _codes(O.N_E4, [[5.0]])          # accumulator holds 15
    assert O.linear_fwd_fp16acc(x8, 3, w8, 1).f64[0, 0] == 15.0 / 16.0
    assert O.linear_fwd_fp16acc(x8, 20, w8, 8).f64[0, 0] == float(np.float16(15.0 * 2.0 ** -28))   # subnormal: rounds
    assert O.linear_fwd_fp16acc(x8, 30, w8, 10).f64[0, 0] == 0.0
    assert np.isinf(O.linear_fwd_fp16acc(x8, -10, w8, -4).f64[0, 0])                                  # 15 * 2^14 > 65504


def test_margin_keeps_the_backward_matmuls_inside_fp16():
    """Section 3.2: FP8-AMAX puts the largest E5 value next to FP16's maximum, so adding two such products overflows
    an FP16 accumulator; a margin of 3 on the gradient's bias leaves room.  dY has two large entries in one row, the
    matching weights are 1."""
    g = np.array([[1.5e-3, 1.4e-3, 1e-6, -2e-6]], dtype=np.float32)
    w = np.array([[1.0, 0.5], [1.0, 0.25], [0.5, 0.125], [0.25, 1.0]], dtype=np.float32)       # W[N=4, K=2]
    _, bw, w8 = O.quantise(w, O.E4)
    assert bw == 7                                    # amax 1 -> bias 7, scaled weights up to 128 (native 256)
    # without a margin the scaled gradient's maximum lands in FP16's top binade
    _, bg0, g8_0 = O.quantise(g, O.E5, margin=0)
    assert O.decode(O.N_E5, int(g8_0[0, 0])) >= 32768.0
    no_margin = O.linear_dgrad_fp16acc(g8_0, bg0, w8, bw + 1, chunk=1)
    assert no_margin.overflowed[0, 0]                 # (49152 * 256 already exceeds 65504)
    # the FP32-accumulate definition of the same product is finite, and a margin alone is not enough when the
    # other operand is scaled to its own maximum: the accumulator holds the product of BOTH scaled operands
    assert np.isfinite(O.linear_dgrad(g8_0, bg0, w8, bw + 1).f64).all()
    # weights of modest scaled size (bias chosen so that the largest scaled weight is 1): now only the E5 operand
    # decides, as in the paper's account: no margin overflows on the second addition, margin 3 survives
    w8_small = O.cast(w, 0, O.N_E4)
    s0 = O.linear_dgrad_fp16acc(g8_0, bg0, w8_small, 0, chunk=1)
    assert s0.overflowed[0, 0]                        # 49152 + 45056 > 65504
    _, bg3, g8_3 = O.quantise(g, O.E5, margin=3)
    assert bg3 == bg0 - 3
    s3 = O.linear_dgrad_fp16acc(g8_3, bg3, w8_small, 0, chunk=1)
    assert not s3.overflowed.any()
    exact = O.linear_dgrad(g8_3, bg3, w8_small, 0).f64
    assert np.allclose(s3.f64, exact, rtol=2.0 ** -10, atol=0.0)


def test_loss_scaling_rescues_small_gradients_from_fp16_underflow():
    """Section 2.4: with an FP16 output the unscaled gradient can fall into FP16's subnormal range; a constant loss
    scale on dY (Table 8 uses 512 ... 32768) moves it back.  The product itself is computed identically: the FP8
    bytes of dY do not change under a power-of-two loss scale, only its bias does.  (The weights take a constant
    bias of 0 here, FP8-CSCALE, so that the scaled accumulator stays far from FP16's maximum.)"""
    rng = np.random.default_rng(3)
    g = (rng.standard_normal((8, 64)) * 1e-6).astype(np.float32)
    w = (rng.standard_normal((64, 16)) * 0.05).astype(np.float32)
    w8 = O.cast(w, 0, O.N_E4)
    ag, bg, g8 = O.quantise(g, O.E5, margin=3)
    plain = O.linear_dgrad_fp16acc(g8, bg, w8, 0, chunk=16)
    exact = O.linear_dgrad(g8, bg, w8, 0).f64
    assert not plain.overflowed.any()
    loss_scale = 4096.0
    ags, bgs, g8s = O.quantise((g * loss_scale).astype(np.float32), O.E5, margin=3)
    assert np.array_equal(g8s, g8) and bgs == bg - 12
    scaled = O.linear_dgrad_fp16acc(g8s, bgs, w8, 0, chunk=16)
    err_plain = np.abs(plain.f64 - exact).max() / np.abs(exact).max()
    err_scaled = np.abs(scaled.f64 / loss_scale - exact).max() / np.abs(exact).max()
    assert err_plain > 0.02 and err_scaled < 2e-3     # subnormal FP16 outputs keep a few bits; scaled ones all eleven


def test_three_matmul_kinds_share_the_index_patterns_of_the_fp32_definitions():
    rng = np.random.default_rng(5)
    T, K, N = 6, 40, 9
    x8 = _codes(O.N_E4, rng.integers(-3, 4, size=(T, K)).astype(float))
    w8 = _codes(O.N_E4, rng.integers(-3, 4, size=(N, K)).astype(float))
    g8 = _codes(O.N_E5, rng.integers(-3, 4, size=(T, N)).astype(float))
    assert np.array_equal(O.linear_fwd_fp16acc(x8, 1, w8, 2, chunk=8).f64, O.linear_fwd(x8, 1, w8, 2).f64)
    assert np.array_equal(O.linear_dgrad_fp16acc(g8, 0, w8, 2, chunk=4).f64, O.linear_dgrad(g8, 0, w8, 2).f64)
    assert np.array_equal(O.linear_wgrad_fp16acc(g8, 0, x8, 1, chunk=3).f64, O.linear_wgrad(g8, 0, x8, 1).f64)
