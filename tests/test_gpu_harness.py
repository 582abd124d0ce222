"""GPU checks of the stress stack's element-wise kernels (include/fp8_harness.h) against the oracle's float64 mirrors
(oracle/stack.py, themselves pinned to torch's float64 GELU and autograd on CPU)."""
import numpy as np
import pytest
import torch

from helpers import bf16_ordinal, bits_of
from oracle import stack as OS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2309_17224_b200 import fp8lin
    return fp8lin


def _every_finite_bf16():
    bits = np.arange(0, 0x10000, dtype=np.uint32).astype(np.uint16)
    bits = bits[(bits & 0x7FFF) < 0x7F80]
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).cuda(), bits


def _ulps(got_bits, want_bits):
    return np.abs(bf16_ordinal(got_bits).astype(np.int64) - bf16_ordinal(want_bits).astype(np.int64))


def test_gelu_for_every_finite_bf16_input(lib):
    x, bits = _every_finite_bf16()
    y = torch.empty_like(x)
    lib.harness_gelu(x, y)
    want = OS.gelu_bits(bits.reshape(1, -1))[0]
    got = bits_of(y.view(1, -1))[0]
    finite = np.abs(OS.bf16_to_f64(want)) < 3.0e38      # the largest inputs overflow bf16 on both sides
    assert _ulps(got[finite], want[finite]).max() <= 1
    assert (got == want).mean() > 0.99


def test_gelu_backward_for_every_finite_bf16_pre_activation(lib):
    pre, bits = _every_finite_bf16()
    for gval in (1.0, -0.37109375, 3.0e-5):
        g = torch.full_like(pre, gval)
        out = torch.empty_like(pre)
        lib.harness_gelu_backward(g, pre, out)
        gv = float(torch.tensor(gval, dtype=torch.bfloat16))
        exact = gv * OS.gelu_grad(bits.reshape(1, -1))[0]
        want = OS.f64_to_bf16(exact)
        got = bits_of(out.view(1, -1))[0]
        # Phi(z) + z phi(z) passes through zero near z = -0.75: there the FP32 sum of two terms of 0.23 keeps an absolute
        # accuracy of a few 2^-24, not a relative one; elsewhere the result is within one bf16 step
        near_root = np.abs(OS.bf16_to_f64(got) - exact) <= abs(gv) * 2.0 ** -21
        assert ((_ulps(got, want) <= 1) | near_root).all()
        assert (_ulps(got, want) <= 1).mean() > 0.999


@pytest.mark.parametrize("n,offset", [(1, 0), (7, 0), (4096 * 1024, 0), (100003, 1), (65537, 3)])
def test_mse_gradient_and_sgd_any_length_and_alignment(lib, n, offset):
    gen = torch.Generator(device="cuda").manual_seed(n)
    base = lambda scale: (torch.randn(n + offset, device="cuda", generator=gen) * scale).to(torch.bfloat16)[offset:]
    y, t = base(1.0), base(1.0)
    g = torch.empty(n + offset, dtype=torch.bfloat16, device="cuda")[offset:]
    scale = 2.0 / n
    lib.harness_mse_grad(y, t, scale, g)
    want = ((y.double() - t.double()) * float(np.float32(scale))).float().to(torch.bfloat16)
    assert _ulps(bits_of(g.view(1, -1))[0], bits_of(want.view(1, -1))[0]).max() <= 1     # one FP32 rounding apart at most
    w32 = torch.randn(n, device="cuda", generator=gen) * 0.02
    dw = base(1e-3)
    w16 = torch.empty(n + offset, dtype=torch.bfloat16, device="cuda")[offset:]
    lr = 1e-3
    want32 = (w32.double() - float(np.float32(lr)) * dw.double()).float()
    lib.harness_sgd(w32, dw, lr, w16)
    assert torch.equal(w32, want32)                       # one fused multiply-add: the correctly rounded result
    assert torch.equal(w16.view(torch.int16), want32.to(torch.bfloat16).view(torch.int16))


def test_harness_argument_errors(lib):
    x = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    raw = lib.raw()
    assert raw.fp8h_gelu(None, x.data_ptr(), 8, None) == lib.ERR_NULL
    assert raw.fp8h_gelu(x.data_ptr(), x.data_ptr(), 0, None) == lib.ERR_SHAPE
    assert raw.fp8h_sgd(None, x.data_ptr(), 0.1, x.data_ptr(), 8, None) == lib.ERR_NULL
