"""Failure detection without a fault: a device-side wait is made to run out, the
kernel returns in an orderly way, the sticky status says so, and the context
keeps working.  Plus guard zones around matmul outputs of ragged shapes."""
import time

import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_bf16_within_one_ulp, bits_of
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


def test_an_expired_wait_is_reported_and_survived(ctx, lib):
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    t0 = time.perf_counter()
    ctx.selftest_wait_expiry(2_000_000)            # 2 ms limit on a barrier nothing completes
    assert time.perf_counter() - t0 < 1.0
    flags = lib.ctypes.c_uint(0)
    st = lib.raw().fp8_device_flags(ctx._h, None, lib.byref(flags), 0)
    assert st == lib.ERR_DEVICE_TIMEOUT and flags.value & lib.FLAG_TIMEOUT
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT   # sticky until cleared
    assert ctx.device_flags() == 0
    # the context and the device are fine: run the real path
    x = torch.randn((256, 512), device="cuda").to(torch.bfloat16)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.amax(x, amax)
    assert float(amax.item()) == float(x.float().abs().max().item())
    with pytest.raises(lib.Fp8Error):
        ctx.selftest_wait_expiry(10 ** 12)         # limits beyond 100 ms are refused


@pytest.mark.parametrize("T,K,N", [(144, 272, 528), (300, 64, 48), (130, 1040, 272), (16, 2048, 48)])
def test_matmuls_write_nothing_outside_their_outputs(ctx, lib, T, K, N):
    """Outputs are carved out of larger buffers; the guard zones on both sides must stay untouched."""
    G = 4096
    x = I.normal_bf16(T, K, 1.0, 3, 1, "cuda")
    w = I.normal_bf16(N, K, 0.02, 3, 2, "cuda")
    g = I.normal_bf16(T, N, 1e-3, 3, 3, "cuda")
    u8k = dict(dtype=torch.uint8, device="cuda")
    sc_f = torch.zeros(3, dtype=torch.float32, device="cuda")
    sc_i = torch.zeros(3, dtype=torch.int32, device="cuda")
    x8, w8, g8 = torch.empty((T, K), **u8k), torch.empty((N, K), **u8k), torch.empty((T, N), **u8k)
    ctx.cast_e4(x, None, d_amax_out=sc_f[0:1], d_bias_out=sc_i[0:1], y=x8)
    ctx.cast_e4(w, None, d_amax_out=sc_f[1:2], d_bias_out=sc_i[1:2], y=w8)
    ctx.cast_e5(g, None, d_amax_out=sc_f[2:3], d_bias_out=sc_i[2:3], y=g8)
    bx, bw, bg = (int(v) for v in sc_i.tolist())
    for dt in (torch.bfloat16, torch.float32):
        outs = {}
        for name, shape in (("y", (T, N)), ("dx", (T, K)), ("dw", (N, K))):
            buf = torch.full((2 * G + shape[0] * shape[1],), 7.0, dtype=dt, device="cuda")
            outs[name] = (buf, buf[G:G + shape[0] * shape[1]].view(shape))
        ctx.linear_fwd(x8, sc_i[0:1], w8, sc_i[1:2], outs["y"][1])
        ctx.linear_dgrad(g8, sc_i[2:3], w8, None, sc_i[1:2], outs["dx"][1])
        ctx.linear_wgrad(g8, None, sc_i[2:3], x8, None, sc_i[0:1], outs["dw"][1], T)
        assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
        for buf, view in outs.values():
            n = view.numel()
            assert bool((buf[:G] == 7.0).all()) and bool((buf[G + n:] == 7.0).all())
        if dt == torch.bfloat16:
            x8h, w8h, g8h = (t.cpu().numpy() for t in (x8, w8, g8))
            assert_bf16_within_one_ulp(bits_of(outs["y"][1]), O.linear_fwd_np(x8h, bx + 1, w8h, bw + 1))
            assert_bf16_within_one_ulp(bits_of(outs["dx"][1]), O.linear_dgrad_np(g8h, bg, w8h, bw + 1))
            assert_bf16_within_one_ulp(bits_of(outs["dw"][1]), O.linear_wgrad_np(g8h, bg, x8h, bx + 1))


def test_launch_count_counts_what_a_call_enqueues(ctx, lib):
    """fp8_launch_count: two launches for amax + cast of a large tensor, one for a decode-size one, one for a cast
    under a given bias, one or two for a matmul (two when the contraction is split through memory)."""
    x = torch.randn(2048, 1024, device="cuda").to(torch.bfloat16)
    small = torch.randn(4, 1024, device="cuda").to(torch.bfloat16)
    y, ys = torch.empty((2048, 1024), dtype=torch.uint8, device="cuda"), torch.empty((4, 1024), dtype=torch.uint8, device="cuda")
    a = torch.zeros(1, dtype=torch.float32, device="cuda")
    b = torch.zeros(1, dtype=torch.int32, device="cuda")
    def span(fn):
        n0 = lib.launch_count()
        fn()
        return lib.launch_count() - n0
    assert span(lambda: ctx.cast_e4(x, None, d_amax_out=a, d_bias_out=b, y=y)) == 2
    assert span(lambda: ctx.cast_e4(small, None, d_amax_out=a, d_bias_out=b, y=ys)) == 1
    assert span(lambda: ctx.cast_e4(x, b, y=y)) == 1
    assert span(lambda: ctx.amax(x, a)) == 1
    w8 = torch.zeros((1024, 1024), dtype=torch.uint8, device="cuda")
    out = torch.empty((2048, 1024), dtype=torch.bfloat16, device="cuda")
    assert span(lambda: ctx.linear_fwd(y, b, w8, b, out)) == 1
    w_long = torch.zeros((512, 8192), dtype=torch.uint8, device="cuda")
    x_long = torch.zeros((4, 8192), dtype=torch.uint8, device="cuda")
    out2 = torch.empty((4, 512), dtype=torch.bfloat16, device="cuda")
    # few tiles, long contraction: the contraction is split; one launch when the slices of a tile meet inside a
    # cluster, two when the partial sums go through memory and a second kernel adds them
    assert span(lambda: ctx.linear_fwd(x_long, b, w_long, b, out2)) in (1, 2)
    # the CTA-pair kernel splits too when tiles are few and the contraction is very long
    x_pair = torch.zeros((512, 16384), dtype=torch.uint8, device="cuda")
    w_pair = torch.zeros((512, 16384), dtype=torch.uint8, device="cuda")
    out3 = torch.empty((512, 512), dtype=torch.bfloat16, device="cuda")
    assert span(lambda: ctx.linear_fwd(x_pair, b, w_pair, b, out3)) == 2
    torch.cuda.synchronize()
