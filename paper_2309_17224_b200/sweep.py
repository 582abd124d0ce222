"""Micro-benchmarks of single entry points (CUDA-event timing, one GPU).

    python -m paper_2309_17224_b200.sweep gemm 8192x8192x16384 8192x8192x4096    # MxNxK forward matmuls
    python -m paper_2309_17224_b200.sweep cast 8192x4096 8192x22016               # amax, cast, amax+cast of bf16 [rows x cols]

Prints one line per shape.  Operands of the matmul sweep are random FP8 bytes
(no NaN codes); a 512 MB buffer is written between cast timings to flush L2.
"""
from __future__ import annotations

import sys

import torch

from . import fp8lin


def _time(fn, iters, pre=None):
    fn()   # first launch of a kernel pays its one-time load
    torch.cuda.synchronize()
    total = 0.0
    for _ in range(iters):
        if pre:
            pre()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        fn()
        e.record()
        torch.cuda.synchronize()
        total += s.elapsed_time(e)
    return total / iters


def gemm(ctx, shapes, iters=20):
    for M, N, K in shapes:
        a = torch.randint(0, 0x78, (M, K), dtype=torch.uint8, device="cuda")
        b = torch.randint(0, 0x78, (N, K), dtype=torch.uint8, device="cuda")
        bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            ctx.linear_fwd(a, bias, b, bias, y)
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(iters):
            ctx.linear_fwd(a, bias, b, bias, y)
        e.record()
        torch.cuda.synchronize()
        ms = s.elapsed_time(e) / iters
        print(f"gemm M={M} N={N} K={K}: {2.0 * M * N * K / ms / 1e9:8.1f} TFLOP/s  {ms * 1e3:8.1f} us", flush=True)


def cast(ctx, shapes, iters=10):
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for rows, cols in shapes:
        x = torch.randn(rows, cols, device="cuda").to(torch.bfloat16)
        n = rows * cols
        amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        y = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
        yt = torch.empty((cols, rows), dtype=torch.uint8, device="cuda")
        ctx.amax(x, amax)
        ctx.scaling_bias(amax, fp8lin.E4, fp8lin.CONV_PAPER, 0, bias)
        fl = flush.zero_
        t_amax = _time(lambda: ctx.amax(x, amax), iters, fl)
        t_flat = _time(lambda: ctx.cast_e4(x, bias, y=y), iters, fl)
        t_both = _time(lambda: ctx.cast_e4(x, bias, y=y, y_t=yt), iters, fl)
        t_fused = _time(lambda: ctx.cast_e4(x, None, d_amax_out=amax, d_bias_out=bias, y=y), iters, fl)
        print(f"cast {rows}x{cols} ({2 * n / 1e6:.0f} MB): amax {t_amax * 1e3:6.1f} us ({2 * n / t_amax / 1e9:5.2f} TB/s)"
              f" | cast {t_flat * 1e3:6.1f} us ({3 * n / t_flat / 1e9:5.2f} TB/s)"
              f" | cast+transposed copy {t_both * 1e3:6.1f} us ({4 * n / t_both / 1e9:5.2f} TB/s)"
              f" | amax+bias+cast {t_fused * 1e3:6.1f} us ({3 * n / t_fused / 1e9:5.2f} TB/s on 3 B/element)", flush=True)


def main(argv):
    if len(argv) < 2 or argv[0] not in ("gemm", "cast"):
        print(__doc__)
        return 2
    shapes = [tuple(int(v) for v in a.split("x")) for a in argv[1:]]
    ctx = fp8lin.Context(0)
    (gemm if argv[0] == "gemm" else cast)(ctx, shapes)
    flags = ctx.device_flags()
    if flags & fp8lin.FLAG_TIMEOUT:
        print("a device-side wait expired", file=sys.stderr)
        return 3
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
