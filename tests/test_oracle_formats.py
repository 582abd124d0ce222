"""Pins for the oracle's FP8 codec: nothing here calls the CUDA library.

The oracle's decode/encode are checked against things fixed outside of it:
Table 7's printed constants, exhaustive code round trips, a numpy brute-force
nearest-value search, torch's own CPU float8 conversions, and byte patterns
worked out by hand from the format definitions.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

FORMATS = {"E4a": O.P_E4, "E5a": O.P_E5, "E4b": O.N_E4, "E5b": O.N_E5}


def _table7(golden_dir):
    rows = {}
    with open(os.path.join(golden_dir, "table7_formats.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, E, M, emax, emin, mx, mn, bias = line.split()
            rows[name] = dict(E=int(E), M=int(M), emax=int(emax), emin=int(emin), max=float(mx),
                              min_sub=float(mn), bias=int(bias))
    return rows


def _finite(fmt):
    t = O.decode_table(fmt)
    return t, np.isfinite(t)


def test_table7_closed_forms(golden_dir):
    t7 = _table7(golden_dir)
    for name, fmt in FORMATS.items():
        row = t7[name]
        table, fin = _finite(fmt)
        mags = table[:128][fin[:128]]
        assert mags.max() == row["max"] == O.max_num(fmt)
        # the closed forms behind the printed columns
        assert row["max"] == (2.0 - 2.0 ** -row["M"] * (2 if name == "E4b" else 1)) * 2.0 ** row["emax"]
        min_sub = mags[mags > 0].min()
        assert min_sub == 2.0 ** (row["emin"] - row["M"])
        # printed with two significant digits
        assert abs(min_sub - row["min_sub"]) <= 0.05 * 10 ** math.floor(math.log10(row["min_sub"]))
        # smallest normal = 2^min_exp sits at exponent field 1
        assert O.decode(fmt, 1 << row["M"]) == 2.0 ** row["emin"]
        # exponent bias: code with exponent field == bias and zero mantissa is 1.0
        assert O.decode(fmt, row["bias"] << row["M"]) == 1.0


def test_finite_code_counts_and_specials():
    counts = {O.P_E4: 255, O.P_E5: 255, O.N_E4: 254, O.N_E5: 248}
    for fmt, n in counts.items():
        _, fin = _finite(fmt)
        assert int(fin.sum()) == n
    # the (a) formats spend the negative-zero code on the single NaN/inf
    assert math.isnan(O.decode(O.P_E4, 0x80)) and math.isnan(O.decode(O.P_E5, 0x80))
    # native E4: only S.1111.111 is NaN; native E5: IEEE inf and NaN
    assert math.isnan(O.decode(O.N_E4, 0x7F)) and math.isnan(O.decode(O.N_E4, 0xFF))
    assert O.decode(O.N_E4, 0x7E) == 448.0 and O.decode(O.N_E4, 0x80) == 0.0
    assert O.decode(O.N_E5, 0x7C) == math.inf and O.decode(O.N_E5, 0xFC) == -math.inf
    assert all(math.isnan(O.decode(O.N_E5, c)) for c in (0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF))


def test_decode_monotonic_and_symmetric():
    for fmt in FORMATS.values():
        table, fin = _finite(fmt)
        mags = [table[c] for c in range(128) if fin[c]]
        assert all(b > a for a, b in zip(mags, mags[1:]))
        for c in range(1, 128):
            if fin[c] and fin[c | 0x80]:
                assert table[c | 0x80] == -table[c]


def test_decode_matches_torch_float8_tables():
    """torch's float8 dtypes are the native (b) formats: an independent decode."""
    codes = torch.arange(256, dtype=torch.uint8)
    for fmt, dt in ((O.N_E4, torch.float8_e4m3fn), (O.N_E5, torch.float8_e5m2)):
        ref = codes.view(dt).to(torch.float64).numpy()
        mine = O.decode_table(fmt)
        assert np.array_equal(np.isnan(ref), np.isnan(mine))
        ok = ~np.isnan(ref)
        assert np.array_equal(ref[ok], mine[ok])
        assert np.array_equal(np.signbit(ref[ok]), np.signbit(mine[ok]))


def test_round_trip_all_codes():
    for fmt in FORMATS.values():
        table, fin = _finite(fmt)
        for c in range(256):
            if fin[c]:
                assert O.encode(fmt, table[c]) == c, (fmt, hex(c))


def test_midpoints_tie_to_even_and_neighbours_round_to_nearest():
    for fmt in FORMATS.values():
        table, fin = _finite(fmt)
        codes = [c for c in range(128) if fin[c]]
        for lo, hi in zip(codes, codes[1:]):
            a, b = table[lo], table[hi]
            mid = 0.5 * (a + b)  # exact in double
            even = lo if lo % 2 == 0 else hi
            assert O.encode(fmt, mid) == even
            assert O.encode(fmt, np.nextafter(mid, 0.0)) == lo
            assert O.encode(fmt, np.nextafter(mid, np.inf)) == hi
            if lo != 0:  # the (a) formats have no negative zero to land on
                assert O.encode(fmt, -mid) == (even | 0x80)


def test_hand_worked_bytes():
    # native E4 (bias 7): 1.0 = 2^0 -> exponent field 7, mantissa 0 -> 0 0111 000
    e4 = {1.0: 0x38, 17.0: 0x58, 19.0: 0x5A, 448.0: 0x7E, 464.0: 0x7E, 480.0: 0x7E, 1e9: 0x7E,
          2.0 ** -9: 0x01, 2.0 ** -10: 0x00, 3 * 2.0 ** -10: 0x02, -2.0 ** -11: 0x80, -1.0: 0xB8}
    for v, c in e4.items():
        assert O.encode(O.N_E4, v) == c, v
    e5 = {57344.0: 0x7B, 61440.0: 0x7B, 1e9: 0x7B, 1.125: 0x3C, 1.375: 0x3E, 2.0 ** -16: 0x01,
          2.0 ** -17: 0x00, 3 * 2.0 ** -17: 0x02, 5 * 2.0 ** -17: 0x02, math.inf: 0x7B, -math.inf: 0xFB}
    for v, c in e5.items():
        assert O.encode(O.N_E5, v) == c, v
    p4 = {240.0: 0x7F, 232.0: 0x7E, 233.0: 0x7F, 1e6: 0x7F, 2.0 ** -10: 0x01, 1.0: 0x40, -2.0 ** -12: 0x00}
    for v, c in p4.items():
        assert O.encode(O.P_E4, v) == c, v
    assert math.isnan(O.decode(O.N_E4, O.encode(O.N_E4, math.nan)))
    assert math.isnan(O.decode(O.N_E5, O.encode(O.N_E5, math.nan)))
    assert O.encode(O.P_E4, math.nan) == 0x80


def _all_bf16_bits():
    return np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(256, 256)


def _bf16_values(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


@pytest.mark.parametrize("fmt,dt,mx", [(O.N_E4, torch.float8_e4m3fn, 448.0), (O.N_E5, torch.float8_e5m2, 57344.0)])
def test_cast_matches_torch_cpu_float8_in_range(fmt, dt, mx):
    """Independent library routine: torch's CPU float8 conversion rounds to
    nearest even on the same grid.  It does not saturate, so compare only
    where the scaled value is finite and within the format's range."""
    bits = _all_bf16_bits()
    x = _bf16_values(bits).to(torch.float32)
    for shift in (-9, -3, 0, 1, 4, 11):
        scaled = x * (2.0 ** shift)  # exact: a power-of-two scaling of an 8-bit significand
        ref = scaled.to(dt).view(torch.uint8).numpy()
        mine = O.cast(bits, shift, fmt)
        ok = (torch.isfinite(scaled) & (scaled.abs() <= mx) & (scaled.abs() >= 2.0 ** -100)).numpy()
        assert ok.sum() > 20000
        assert np.array_equal(ref[ok], mine[ok])


@pytest.mark.parametrize("fmt", [O.N_E4, O.N_E5, O.P_E4, O.P_E5])
def test_cast_is_a_nearest_value_search(fmt):
    """Brute force with numpy on the (already pinned) decode table: the chosen
    code is a closest value, and on a tie it is the even code."""
    table, fin = _finite(fmt)
    mag_codes = np.array([c for c in range(128) if fin[c]])
    mags = table[mag_codes]
    bits = _all_bf16_bits()
    vals = _bf16_values(bits).to(torch.float64).numpy()
    for shift in (-140, -20, -2, 0, 3, 9, 40, 135):
        got = O.cast(bits, shift, fmt)
        v = np.ldexp(vals, shift)
        finite = np.isfinite(v)
        a = np.abs(v[finite])
        g = got[finite]
        d = np.abs(mags[None, :] - a[:, None])
        best = d.min(axis=1)
        chosen = table[g & 0x7F]
        clipped = a >= mags.max()
        assert np.all(chosen[clipped] == mags.max())
        assert np.all(np.abs(chosen[~clipped] - a[~clipped]) == best[~clipped])
        ties = (d == best[:, None]).sum(axis=1) > 1
        assert np.all((g[ties & ~clipped] & 1) == 0)
        # sign: kept on every non-zero result; native formats keep it on zero too
        neg = np.signbit(v[finite])
        if fmt in (O.N_E4, O.N_E5):
            assert np.array_equal((g >> 7).astype(bool), neg)
        else:
            nz = (g & 0x7F) != 0
            assert np.array_equal((g[nz] >> 7).astype(bool), neg[nz])
            assert not np.any(g == 0x80)
        # infinities clip, NaNs become the format's NaN
        inf = np.isinf(v)
        assert np.all(table[got[inf] & 0x7F] == mags.max())
        nan = np.isnan(v)
        assert np.all(np.isnan(table[got[nan]]))


def test_transposed_copy_holds_the_same_codes():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 65536, size=(37, 53), dtype=np.uint32).astype(np.uint16)
    y, y_t = O.cast(bits, 2, O.N_E4, transposed=True)
    assert y.shape == (37, 53) and y_t.shape == (53, 37)
    assert np.array_equal(y.T, y_t)


def test_paper_and_native_bytes_are_linked_by_the_documented_shift():
    """E4: a paper byte read as a native byte is exactly twice the value, apart
    from +-240 (natively NaN) and the paper's NaN code (natively -0).
    E5: equal values, exponent field one lower, apart from the odd multiples of
    2^-17 below 2^-14 that the native grid does not have."""
    p4, n4 = O.decode_table(O.P_E4), O.decode_table(O.N_E4)
    for c in range(256):
        if c in (0x7F, 0xFF, 0x80):
            continue
        assert n4[c] == 2.0 * p4[c]
    p5, n5 = O.decode_table(O.P_E5), O.decode_table(O.N_E5)
    unmapped = []
    for c in range(256):
        if c == 0x80:
            continue
        v = p5[c]
        back = O.decode(O.N_E5, O.encode(O.N_E5, v))
        if back != v:
            unmapped.append(c)
        elif (c & 0x7F) >= 8:
            assert O.encode(O.N_E5, v) == c - 4
    assert unmapped == [0x01, 0x03, 0x05, 0x07, 0x81, 0x83, 0x85, 0x87]
    assert [O.encode(O.N_E5, p5[c]) for c in (2, 4, 6)] == [1, 2, 3]


def test_casting_with_the_shifted_bias_reproduces_the_paper_format_bytes():
    """Casting x*2^b to the paper's E4 and x*2^(b+1) to native E4 gives the
    same byte except where the paper byte has no native counterpart."""
    bits = _all_bf16_bits()
    for b in (-6, -1, 0, 2, 7, 15):
        paper = O.cast(bits, b, O.P_E4)
        native = O.cast(bits, b + 1, O.N_E4)
        vals = np.ldexp(_bf16_values(bits).to(torch.float64).numpy(), b)
        differ = paper != native
        for pc, nc, v in zip(paper[differ], native[differ], vals[differ]):
            if pc in (0x7F, 0xFF):          # +-240 saturates one step lower natively
                assert nc == pc - 1
            elif pc == 0x00:                # negative underflow keeps its sign natively
                assert nc == 0x80 and np.signbit(v)
            elif pc == 0x80:                # NaN
                assert np.isnan(v) and nc in (0x7F, 0xFF)
            else:
                raise AssertionError((hex(pc), hex(nc), v))
