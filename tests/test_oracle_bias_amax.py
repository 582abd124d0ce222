"""Pins for the oracle's amax and scaling bias (Eq. 3): hand values, exact
rational arithmetic over every bf16 value, the defining inequality."""
from fractions import Fraction

import numpy as np
import torch

import oracle as O


def test_hand_computed_biases():
    # (amax, E4 with max 240, E4 with max 448, E5 with max 57344)
    hand = [
        (240.0, 0, 0, 7),        # 240*2^0 = 240 fits exactly; 240*2 = 480 > 448; 240*2^7 = 30720 <= 57344 < 61440
        (241.0, -1, 0, 7),
        (120.0, 1, 1, 8),
        (1.0, 7, 8, 15),         # 2^7 <= 240 < 2^8; 2^8 <= 448 < 2^9; 2^15 <= 57344 < 2^16
        (1.875, 7, 7, 14),       # 1.875*2^7 = 240 exactly
        (1.8828125, 6, 7, 14),   # next bf16 after 1.875 no longer fits at 2^7
        (5.0, 5, 6, 13),
        (0.08, 11, 12, 19),
        (0.005, 15, 16, 23),
        (57344.0, -8, -7, 0),
    ]
    for amax, b4p, b4n, b5 in hand:
        assert O.scaling_bias(amax, O.E4, O.CONV_PAPER) == b4p, amax
        assert O.scaling_bias(amax, O.E4, O.CONV_NATIVE) == b4n, amax
        assert O.scaling_bias(amax, O.E5, O.CONV_PAPER) == b5, amax
        assert O.scaling_bias(amax, O.E5, O.CONV_NATIVE) == b5, amax


def test_margin_is_subtracted():
    assert O.scaling_bias(1.0, O.E5, O.CONV_PAPER, margin=3) == 12
    assert O.scaling_bias(1.0, O.E4, O.CONV_PAPER, margin=-2) == 9


def test_degenerate_amax():
    assert O.scaling_bias(0.0, O.E4) == 0
    assert O.scaling_bias(float("inf"), O.E4) == 0
    assert O.scaling_bias(float("nan"), O.E5) == 0


def test_bias_is_floor_log2_for_every_bf16_amax():
    """floor(log2(max_num/amax)) evaluated in exact rational arithmetic for all
    32 639 positive finite bf16 values, plus the inequality that defines it."""
    bits = np.arange(1, 0x7F80, dtype=np.uint32).astype(np.uint16)
    vals = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    ranges = {}
    for kind, conv, mx in ((O.E4, O.CONV_PAPER, 240), (O.E4, O.CONV_NATIVE, 448), (O.E5, O.CONV_PAPER, 57344)):
        lo, hi = 10 ** 9, -10 ** 9
        for v in vals.tolist():
            a = Fraction(v)
            b = O.scaling_bias(v, kind, conv)
            two_b = Fraction(2) ** b
            assert a * two_b <= mx < a * two_b * 2, (v, b)
            lo, hi = min(lo, b), max(hi, b)
        ranges[(kind, conv)] = (lo, hi)
    # extreme biases reached at the largest / smallest bf16 magnitudes
    assert ranges[(O.E4, O.CONV_PAPER)] == (-121, 140)
    assert ranges[(O.E4, O.CONV_NATIVE)] == (-120, 141)
    assert ranges[(O.E5, O.CONV_PAPER)] == (-113, 148)


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def test_amax_against_numpy_and_special_values():
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(33, 70, generator=g) * 3).to(torch.bfloat16)
    assert O.amax(_bits(x)) == float(x.to(torch.float64).abs().max())
    x[5, 6] = -1000.0
    assert O.amax(_bits(x)) == 1000.0
    x[7, 1] = float("inf")
    assert O.amax(_bits(x)) == float("inf")
    x[0, 0] = float("nan")
    assert np.isnan(O.amax(_bits(x)))
    z = torch.zeros(4, 4, dtype=torch.bfloat16)
    z[1, 1] = -0.0
    assert O.amax(_bits(z)) == 0.0
    # a bf16 subnormal
    s = np.zeros((2, 2), dtype=np.uint16)
    s[1, 0] = 0x8001
    assert O.amax(s) == 2.0 ** -133


def test_scaling_a_tensor_by_a_power_of_two_moves_only_the_bias():
    g = torch.Generator().manual_seed(4)
    x = torch.randn(40, 24, generator=g).to(torch.bfloat16)
    a0, b0, y0 = O.quantise(_bits(x), O.E4)
    for k in (-9, 5):
        xk = (x.to(torch.float32) * 2.0 ** k).to(torch.bfloat16)
        ak, bk, yk = O.quantise(_bits(xk), O.E4)
        assert ak == a0 * 2.0 ** k and bk == b0 - k
        assert np.array_equal(yk, y0)


def test_largest_cast_code_lands_in_the_top_binade():
    """After scaling by the AMAX bias the largest element sits in
    [max_num/2, max_num] of the format Eq. 3 was evaluated for."""
    g = torch.Generator().manual_seed(5)
    for std in (1e-4, 0.02, 1.0, 300.0):
        x = (torch.randn(64, 64, generator=g) * std).to(torch.bfloat16)
        for kind, conv in ((O.E4, O.CONV_PAPER), (O.E4, O.CONV_NATIVE), (O.E5, O.CONV_PAPER)):
            a, b, y = O.quantise(_bits(x), kind, conv)
            top = np.abs(O.decode_table(O.native_format(kind))[y]).max() * 2.0 ** -O.delta(kind, conv)
            mx = O.bias_max_num(kind, conv)
            assert mx / 2 <= top <= mx or (conv == O.CONV_PAPER and kind == O.E4 and top == 224.0)


def test_fp16_and_fp32_inputs_are_read_exactly():
    """Every fp16 bit pattern decodes as numpy decodes it; amax and cast on
    fp16 / fp32 tensors equal the same operations on the exactly converted
    bf16-free reference path (numpy float64 arithmetic + the pinned encoder)."""
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16).view(np.float16).reshape(256, 256)
    finite = np.isfinite(h)
    assert O.amax(np.where(finite, h, np.float16(0))) == float(np.abs(h[finite].astype(np.float64)).max()) == 65504.0
    assert np.isnan(O.amax(h))
    table = O.decode_table(O.N_E4)
    for shift in (-3, 0, 6):
        codes = O.cast(h, shift, O.N_E4)
        v = np.ldexp(h.astype(np.float64), shift)
        ok = finite & (np.abs(v) <= 448.0)
        # the chosen value is a nearest grid value
        grid = table[:0x7F]
        best = np.abs(grid[None, :] - np.abs(v[ok])[:, None]).min(axis=1)
        assert np.array_equal(np.abs(table[codes[ok] & 0x7F] - np.abs(v[ok])), best)
    rng = np.random.default_rng(3)
    f = (rng.standard_normal((64, 48)) * 5).astype(np.float32)
    f[0, 0] = -123.456
    assert O.amax(f) == np.float32(123.456)
    got = O.cast(f, 1, O.N_E4)
    ref = torch.from_numpy(f * 2.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    ok = np.abs(f * 2.0) <= 448.0
    assert np.array_equal(got[ok], ref[ok])


def test_history_bias_is_eq3_on_the_window_maximum():
    """Amax-history scaling: a window of one is the just-in-time bias; for a longer window every entry fits
    under the bias (entry * 2^b <= max_num) while the largest one would not fit under b + 1."""
    from fractions import Fraction
    rng = np.random.default_rng(3)
    for kind, mx in ((O.E4, 240), (O.E5, 57344)):
        for _ in range(50):
            window = [float(np.float32(2.0 ** rng.uniform(-20, 20))) for _ in range(int(rng.integers(1, 9)))]
            assert O.history_bias(window[:1], kind) == O.scaling_bias(window[0], kind)
            b = O.history_bias(window, kind)
            assert all(Fraction(a) * Fraction(2) ** b <= mx for a in window)
            assert Fraction(max(window)) * Fraction(2) ** (b + 1) > mx
            assert O.history_bias(window, kind, O.CONV_PAPER, 3) == b - 3


def test_paper_e4_top_code_has_no_native_byte():
    """Table 7 row (a) puts the E4 maximum at 240; read as a native byte its code is NaN.  A tensor whose scaled
    amax lands in (232, 240] therefore carries 224 (byte 0x7E) for its largest elements under the paper
    convention, and is untouched under the native convention (max_num 448 leaves it one binade of headroom)."""
    for top, want in ((236.0, 0x7E), (240.0, 0x7E), (232.0, 0x7E), (231.0, 0x7E), (228.0, 0x7E), (216.0, 0x7E),
                      (215.0, 0x7D)):
        x = np.array([[top, -top, 1.0, 0.5]], dtype=np.float32)
        a, b, y = O.quantise(x, O.E4, O.CONV_PAPER)
        assert (a, b) == (top, 0)
        assert y[0, 0] == want and y[0, 1] == (want | 0x80)
    # what the byte means in paper units: native value / 2
    assert O.decode(O.N_E4, 0x7E) / 2 == 224.0
    a, b, y = O.quantise(np.array([[236.0, 1.0]], dtype=np.float32), O.E4, O.CONV_NATIVE)
    assert b == 0 and O.decode(O.N_E4, int(y[0, 0])) == 240.0   # 236 rounds to 240 on the native grid, no clipping


def test_bias_mode_of_hand_made_sequences():
    """Appendix G's per-tensor statistic: the most frequent bias; the smaller value on a tie."""
    assert O.bias_mode([7, 7, 6, 7, 8, 6]) == (7, 3)
    assert O.bias_mode([5, 6, 6, 5]) == (5, 2)            # tie -> smaller
    assert O.bias_mode([-3, -4, -4, -3, 2]) == (-4, 2)    # tie between negatives -> smaller
    assert O.bias_mode([19]) == (19, 1)
    assert O.bias_mode([]) == (0, 0)
    # against a library routine on random draws: scipy's mode also returns the smallest of the most frequent values
    from scipy import stats
    rng = np.random.default_rng(4)
    for _ in range(20):
        seq = rng.integers(-6, 7, size=int(rng.integers(1, 40)))
        m = stats.mode(seq, keepdims=False)
        assert O.bias_mode(seq) == (int(m.mode), int(m.count))
