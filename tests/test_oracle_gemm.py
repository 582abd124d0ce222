"""Pins for the oracle's three matmuls and the unscale (Eq. 2, Section 2.2):
an exactly representable worked example, integer matrices against numpy's
integer matmul, numpy float64 matmul on the pinned decode tables, the
power-of-two scale/unscale identity, torch's bf16 rounding."""
import numpy as np
import torch

import oracle as O


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _bf16_from_bits(b):
    return torch.from_numpy(b.view(np.int16).copy()).view(torch.bfloat16)


def test_worked_example_is_exact():
    # X = [[1,-2],[0.5,3]]: amax 3, 3*2^6 = 192 <= 240 < 384 -> b = 6, shift 7:
    # 128, -256, 64, 384 in native E4 = 0x70, 0xF8, 0x68, 0x7C.
    X = torch.tensor([[1.0, -2.0], [0.5, 3.0]], dtype=torch.bfloat16)
    W = torch.tensor([[0.25, 0.5], [-1.0, 0.125]], dtype=torch.bfloat16)
    ax, bx, x8 = O.quantise(_bits(X), O.E4)
    aw, bw, w8 = O.quantise(_bits(W), O.E4)
    assert (ax, bx) == (3.0, 6) and (aw, bw) == (1.0, 7)
    assert x8.tolist() == [[0x70, 0xF8], [0x68, 0x7C]]
    assert w8.tolist() == [[0x68, 0x70], [0xF8, 0x60]]
    res = O.linear_fwd(x8, bx + 1, w8, bw + 1)
    assert res.f64.tolist() == [[-0.75, -1.25], [1.625, -0.125]]
    assert res.f32.tolist() == [[-0.75, -1.25], [1.625, -0.125]]
    assert res.abs_sum.tolist() == [[1.25, 1.25], [1.625, 0.875]]
    assert _bf16_from_bits(res.bf16).float().tolist() == [[-0.75, -1.25], [1.625, -0.125]]


def _int_tensor(rng, rows, cols, hi):
    return torch.from_numpy(rng.integers(-hi, hi + 1, size=(rows, cols)).astype(np.float32)).to(torch.bfloat16)


def test_small_integer_matrices_reproduce_integer_matmul():
    """Integers up to 14 (E4, four significant bits; 15 would scale to the
    paper format's 240, the one magnitude the native format cannot hold) and
    up to 7 (E5) are exactly representable after any power-of-two scaling, so
    the FP8 path must equal the integer product."""
    rng = np.random.default_rng(7)
    T, K, N = 9, 21, 13
    X, W, G = _int_tensor(rng, T, K, 14), _int_tensor(rng, N, K, 14), _int_tensor(rng, T, N, 7)
    Xi, Wi, Gi = (t.to(torch.int64).numpy() for t in (X, W, G))
    _, bx, x8 = O.quantise(_bits(X), O.E4)
    _, bw, w8 = O.quantise(_bits(W), O.E4)
    _, bg, g8 = O.quantise(_bits(G), O.E5)
    sx, sw, sg = bx + 1, bw + 1, bg
    assert np.array_equal(O.linear_fwd(x8, sx, w8, sw).f64, (Xi @ Wi.T).astype(np.float64))
    assert np.array_equal(O.linear_dgrad(g8, sg, w8, sw).f64, (Gi @ Wi).astype(np.float64))
    assert np.array_equal(O.linear_wgrad(g8, sg, x8, sx).f64, (Gi.T @ Xi).astype(np.float64))


def test_against_numpy_matmul_on_decoded_operands():
    rng = np.random.default_rng(8)
    T, K, N = 17, 40, 23
    x8 = rng.integers(0, 0x78, size=(T, K), dtype=np.uint8) | (rng.integers(0, 2, size=(T, K), dtype=np.uint8) << 7)
    w8 = rng.integers(0, 0x78, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7)
    g8 = rng.integers(0, 0x78, size=(T, N), dtype=np.uint8) | (rng.integers(0, 2, size=(T, N), dtype=np.uint8) << 7)
    t4, t5 = O.decode_table(O.N_E4), O.decode_table(O.N_E5)
    X, W, G = t4[x8], t4[w8], t5[g8]
    bias_vec = rng.standard_normal(N)
    sx, sw, sg = 3, -2, 5
    fwd = O.linear_fwd(x8, sx, w8, sw, bias_vec=bias_vec)
    np.testing.assert_allclose(fwd.f64, (X @ W.T) * 2.0 ** -(sx + sw) + bias_vec, rtol=1e-13, atol=0)
    np.testing.assert_allclose(fwd.abs_sum, (np.abs(X) @ np.abs(W).T) * 2.0 ** -(sx + sw) + np.abs(bias_vec), rtol=1e-13)
    dg = O.linear_dgrad(g8, sg, w8, sw)
    np.testing.assert_allclose(dg.f64, (G @ W) * 2.0 ** -(sg + sw), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(dg.abs_sum, (np.abs(G) @ np.abs(W)) * 2.0 ** -(sg + sw), rtol=1e-13)
    wg = O.linear_wgrad(g8, sg, x8, sx)
    np.testing.assert_allclose(wg.f64, (G.T @ X) * 2.0 ** -(sg + sx), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(wg.abs_sum, (np.abs(G).T @ np.abs(X)) * 2.0 ** -(sg + sx), rtol=1e-13)
    # f32 is one rounding of the exact value; bf16 is torch's rounding of that
    assert np.array_equal(fwd.f32, fwd.f64.astype(np.float32))
    assert np.array_equal(_bf16_from_bits(fwd.bf16).float().numpy(),
                          torch.from_numpy(fwd.f32).to(torch.bfloat16).float().numpy())


def test_samples_equal_the_full_product():
    rng = np.random.default_rng(9)
    T, K, N = 11, 19, 14
    x8 = rng.integers(0, 0x78, size=(T, K), dtype=np.uint8)
    w8 = rng.integers(0x80, 0xF8, size=(N, K), dtype=np.uint8)
    g8 = rng.integers(0, 0x78, size=(T, N), dtype=np.uint8)
    bv = rng.standard_normal(N)
    full = {O.FWD: O.linear_fwd(x8, 1, w8, 2, bias_vec=bv), O.DGRAD: O.linear_dgrad(g8, 3, w8, 2),
            O.WGRAD: O.linear_wgrad(g8, 3, x8, 1)}
    ops = {O.FWD: (x8, O.N_E4, 1, w8, O.N_E4, 2), O.DGRAD: (g8, O.N_E5, 3, w8, O.N_E4, 2),
           O.WGRAD: (g8, O.N_E5, 3, x8, O.N_E4, 1)}
    for kind, res in full.items():
        R, C = res.f64.shape
        rows, cols = rng.integers(0, R, 50), rng.integers(0, C, 50)
        s = O.linear_samples(kind, *ops[kind], rows, cols, bias_vec=bv if kind == O.FWD else None)
        assert np.array_equal(s.f64, res.f64[rows, cols])
        assert np.array_equal(s.f32, res.f32[rows, cols])
        assert np.array_equal(s.bf16, res.bf16[rows, cols])
        assert np.array_equal(s.abs_sum, res.abs_sum[rows, cols])


def test_scale_then_unscale_is_a_power_of_two_round_trip():
    """Multiplying an input by 2^k moves its bias by -k, keeps its bytes and
    multiplies the output by exactly 2^k (Eqs. 1 and 2)."""
    g = torch.Generator().manual_seed(11)
    X = torch.randn(12, 32, generator=g).to(torch.bfloat16)
    W = (torch.randn(10, 32, generator=g) * 0.02).to(torch.bfloat16)
    _, bx, x8 = O.quantise(_bits(X), O.E4)
    _, bw, w8 = O.quantise(_bits(W), O.E4)
    base = O.linear_fwd(x8, bx + 1, w8, bw + 1).f32
    k = 6
    Xk = (X.float() * 2.0 ** k).to(torch.bfloat16)
    _, bxk, x8k = O.quantise(_bits(Xk), O.E4)
    assert bxk == bx - k and np.array_equal(x8k, x8)
    assert np.array_equal(O.linear_fwd(x8k, bxk + 1, w8, bw + 1).f32, base * np.float32(2.0 ** k))


def test_fp8_product_stays_close_to_the_bf16_product():
    """Sanity on magnitude and sign conventions: with E4's 3 mantissa bits the
    FP8 result differs from the unquantised product by a few percent of
    sum|x||w| at most."""
    g = torch.Generator().manual_seed(12)
    X = torch.randn(16, 256, generator=g).to(torch.bfloat16)
    W = (torch.randn(24, 256, generator=g) * 0.02).to(torch.bfloat16)
    _, bx, x8 = O.quantise(_bits(X), O.E4)
    _, bw, w8 = O.quantise(_bits(W), O.E4)
    res = O.linear_fwd(x8, bx + 1, w8, bw + 1)
    exact = X.double().numpy() @ W.double().numpy().T
    bound = np.abs(X.double().numpy()) @ np.abs(W.double().numpy()).T
    assert np.all(np.abs(res.f64 - exact) <= 0.13 * bound)
    assert np.corrcoef(res.f64.ravel(), exact.ravel())[0, 1] > 0.99


def test_numpy_matmul_variants_agree_with_the_plain_loops():
    """The float64-BLAS forms against the plain C loops: float64 sums to 2^-50 of sum |a*b| (the order of the
    additions may differ by a rounding of the float64 sum when E5 x E4 terms span more than 53 bits), the FP32 and
    bf16 roundings equal except where that last bit decides a tie (none on these inputs)."""
    rng = np.random.default_rng(21)
    T, K, N = 70, 300, 90
    x8 = rng.integers(0, 0x7F, size=(T, K), dtype=np.uint8) | (rng.integers(0, 2, size=(T, K), dtype=np.uint8) << 7)
    w8 = rng.integers(0, 0x7F, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7)
    g8 = rng.integers(0, 0x7C, size=(T, N), dtype=np.uint8) | (rng.integers(0, 2, size=(T, N), dtype=np.uint8) << 7)
    bv = rng.standard_normal(N)
    pairs = [(O.linear_fwd(x8, 9, w8, -3, bias_vec=bv), O.linear_fwd_np(x8, 9, w8, -3, bias_vec=bv)),
             (O.linear_dgrad(g8, 21, w8, -3), O.linear_dgrad_np(g8, 21, w8, -3)),
             (O.linear_wgrad(g8, 21, x8, 9), O.linear_wgrad_np(g8, 21, x8, 9))]
    for plain, fast in pairs:
        assert np.all(np.abs(plain.f64 - fast.f64) <= 2.0 ** -50 * plain.abs_sum)
        assert np.all(np.abs(plain.abs_sum - fast.abs_sum) <= 2.0 ** -50 * plain.abs_sum)
        assert np.array_equal(plain.f32, fast.f32)
        assert np.array_equal(plain.bf16, fast.bf16)


def test_vectorised_bf16_rounding_is_the_scalar_rule():
    """f32_to_bf16_bits_np against orc_f32_to_bf16 element by element: ties both ways, carries into the exponent,
    overflow to infinity, subnormals, NaN."""
    vals = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2.0 ** -9, 1.0 + 3 * 2.0 ** -9, 3.3895314e38, 3.4e38, 1e-40,
                     -1e-40, 0.0, -0.0, np.inf, -np.inf, np.nan, 65280.0, 65408.0, 65407.99], dtype=np.float32)
    rng = np.random.default_rng(3)
    vals = np.concatenate([vals, rng.standard_normal(2000).astype(np.float32),
                           rng.integers(0, 2 ** 32, 4000, dtype=np.uint64).astype(np.uint32).view(np.float32)])
    a, b = O.f32_to_bf16_bits(vals), O.f32_to_bf16_bits_np(vals)
    nan = np.isnan(vals)
    assert np.array_equal(a[~nan], b[~nan])
    assert np.all((a[nan] & 0x7FFF) > 0x7F80) and np.all((b[nan] & 0x7FFF) > 0x7F80)


def test_sampled_matmul_equals_the_full_product():
    """orc_linear_samples (decode values tabulated once per call) against the full C products, every kind."""
    rng = np.random.default_rng(22)
    T, K, N = 33, 48, 40
    x8 = rng.integers(0, 0x7F, size=(T, K), dtype=np.uint8) | (rng.integers(0, 2, size=(T, K), dtype=np.uint8) << 7)
    w8 = rng.integers(0, 0x7F, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7)
    g8 = rng.integers(0, 0x7C, size=(T, N), dtype=np.uint8) | (rng.integers(0, 2, size=(T, N), dtype=np.uint8) << 7)
    bv = rng.standard_normal(N)
    cases = [(O.FWD, (x8, O.N_E4, 5, w8, O.N_E4, -2), O.linear_fwd(x8, 5, w8, -2, bias_vec=bv), bv),
             (O.DGRAD, (g8, O.N_E5, 11, w8, O.N_E4, -2), O.linear_dgrad(g8, 11, w8, -2), None),
             (O.WGRAD, (g8, O.N_E5, 11, x8, O.N_E4, 5), O.linear_wgrad(g8, 11, x8, 5), None)]
    for kind, ops, full, bias in cases:
        R, C = full.f64.shape
        rows, cols = np.divmod(np.arange(R * C), C)
        s = O.linear_samples(kind, *ops, rows, cols, bias_vec=bias)
        assert np.array_equal(s.f64.reshape(R, C), full.f64) and np.array_equal(s.abs_sum.reshape(R, C), full.abs_sum)
        assert np.array_equal(s.f32.reshape(R, C), full.f32) and np.array_equal(s.bf16.reshape(R, C), full.bf16)
