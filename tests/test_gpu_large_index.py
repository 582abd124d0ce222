"""GPU parity at sizes whose element indices do not fit 32 bits: a tensor of more than 2^31 elements through amax,
bias and cast (both layouts), and a matmul whose output has more than 2^31 elements.  The oracle checks what it can
reach in seconds: the amax planted beyond index 2^31, whole sampled rows / columns of bytes, sampled outputs."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_bf16_within_one_ulp, assert_codes_equal, bits_of, u8

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


def test_amax_and_cast_of_a_tensor_beyond_2_to_the_31_elements(ctx, lib):
    rows, cols = 65600, 32784                       # 2 150 630 400 elements; the last 48 rows lie beyond index 2^31
    assert rows * cols > 2 ** 31 and (rows - 48) * cols > 2 ** 31
    x = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(2309)
    for r0 in range(0, rows, 8200):                 # seeded, in slabs (no 8 GB float32 temporary)
        x[r0:r0 + 8200].copy_(torch.randn((min(8200, rows - r0), cols), generator=g, device="cuda"))
    x[rows - 3, cols - 5] = -77.5                   # the amax sits at linear index > 2^31
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    bias = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    y_t = torch.empty((cols, rows), dtype=torch.uint8, device="cuda")
    ctx.cast_e4(x, None, d_amax_out=amax, d_bias_out=bias, y=y, y_t=y_t)
    assert float(amax.item()) == 77.5
    b = O.scaling_bias(77.5, O.E4)
    assert int(bias.item()) == b
    amax2 = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.amax(x, amax2)
    assert float(amax2.item()) == 77.5
    pick = [0, 1, 32767, 32768, rows - 49, rows - 48, rows - 3, rows - 1]
    want = O.cast(bits_of(x[pick].contiguous()), b + 1, O.N_E4)
    assert_codes_equal(u8(y[pick].contiguous()), want, O.N_E4)
    assert np.array_equal(u8(y_t[:, pick].contiguous()), want.T)
    # the flat (row-major only) path and the one-pass path on the same tensor
    y.zero_()
    ctx.cast_e4(x, bias, y=y)
    assert_codes_equal(u8(y[pick].contiguous()), want, O.N_E4)
    y.zero_()
    ctx.cast_predicted(lib.E4, x, amax2, bias, y)
    assert int(bias.item()) == b
    assert_codes_equal(u8(y[pick].contiguous()), want, O.N_E4)
    assert ctx.device_flags(clear=True) & ~lib.FLAG_SATURATED == 0


def test_matmul_with_more_than_2_to_the_31_outputs(ctx, lib):
    T, N, K = 65792, 33024, 128                     # 2 172 715 008 outputs
    assert T * N > 2 ** 31
    g = torch.Generator(device="cuda").manual_seed(17224)
    x8 = torch.randint(0, 0x78, (T, K), dtype=torch.uint8, device="cuda", generator=g)
    w8 = torch.randint(0, 0x78, (N, K), dtype=torch.uint8, device="cuda", generator=g)
    x8 |= (torch.randint(0, 2, (T, K), dtype=torch.uint8, device="cuda", generator=g) << 7)     # signs
    x8[x8 == 0x80] = 0                              # the paper's formats have no negative zero
    bx = torch.tensor([3], dtype=torch.int32, device="cuda")
    bw = torch.tensor([-2], dtype=torch.int32, device="cuda")
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    amax_y = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.linear_fwd(x8, bx, w8, bw, y, d_amax_y=amax_y)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    rng = np.random.default_rng(5)
    rows = np.concatenate([rng.integers(0, T, 3000), rng.integers(T - 700, T, 1000), [0, T - 1, T - 1, 0]])
    cols = np.concatenate([rng.integers(0, N, 4000), [0, N - 1, 0, N - 1]])
    ref = O.linear_samples(O.FWD, u8(x8), O.N_E4, 3 + 1, u8(w8), O.N_E4, -2 + 1, rows, cols)
    got = y[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()]
    assert_bf16_within_one_ulp(bits_of(got.reshape(1, -1))[0], ref)
    # the emitted amax against a reduction over the whole output, in slabs
    m = 0.0
    for r0 in range(0, T, 8224):
        m = max(m, float(y[r0:r0 + 8224].float().abs().max().item()))
    assert float(amax_y.item()) == m
