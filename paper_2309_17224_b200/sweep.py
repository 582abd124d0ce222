"""Micro-benchmarks of single entry points (CUDA-event timing, one GPU).

    python -m paper_2309_17224_b200.sweep gemm 8192x8192x16384 8192x8192x4096    # MxNxK forward matmuls
    python -m paper_2309_17224_b200.sweep cast 8192x4096 8192x22016               # amax, cast, amax+cast of bf16 [rows x cols]
    python -m paper_2309_17224_b200.sweep stack 24x1024x4096                      # layers x d x tokens: the SGD stack, three scaling variants
    python -m paper_2309_17224_b200.sweep mlp 8192x4096x11008                     # tokens x d x ffn: a Llama MLP forward, unfused vs SwiGLU epilogue
    python -m paper_2309_17224_b200.sweep stack 24x1024x4096 --only history --steps 2 --warmup 2 --no-graph   # one variant, short (for profilers)

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
        line = f"gemm M={M} N={N} K={K}: {2.0 * M * N * K / ms / 1e9:8.1f} TFLOP/s  {ms * 1e3:8.1f} us"
        if N % 16 == 0 and K % 16 == 0:
            # the fused epilogues on the same operands: GELU + amax; GELU + amax + FP8 bytes; GELU' of a stored
            # pre-activation + amax + FP8 bytes (input-gradient matmul, so its output is [M, K])
            z = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            z8 = torch.empty((M, N), dtype=torch.uint8, device="cuda")
            amax = torch.zeros(1, dtype=torch.float32, device="cuda")
            g8 = torch.empty((M, K), dtype=torch.uint8, device="cuda")
            pre = torch.randn((M, K), device="cuda").to(torch.bfloat16)
            dy = torch.randint(0, 0x78, (M, N), dtype=torch.uint8, device="cuda")
            runs = (("gelu", lambda: ctx.linear_fwd_act(a, bias, b, bias, y, z, d_amax_act=amax)),
                    ("gelu->fp8", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias, y_pre=y, d_amax_z=amax,
                                                           act=fp8lin.ACT_GELU)),
                    ("gelu->fp8 (bytes only)", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias, act=fp8lin.ACT_GELU)),
                    ("->fp8 (bytes only)", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias)),
                    ("dgrad gelu'->fp8", lambda: ctx.linear_dgrad_q(dy, bias, b, None, bias, g8, bias, y_pre=pre,
                                                                     d_amax_g=amax, act=fp8lin.ACT_GELU)))
            if N % 64 == 0 and K % 32 == 0:
                zs = torch.empty((M, N // 2), dtype=torch.uint8, device="cuda")
                gs = torch.empty((M, 2 * K), dtype=torch.uint8, device="cuda")
                pre2 = torch.randn((M, 2 * K), device="cuda").to(torch.bfloat16)
                runs += (("swiglu->fp8", lambda: ctx.linear_fwd_q(a, bias, b, bias, zs, bias, y_pre=y, d_amax_z=amax,
                                                                  act=fp8lin.ACT_SWIGLU)),
                         ("dgrad swiglu'->fp8", lambda: ctx.linear_dgrad_q(dy, bias, b, None, bias, gs, bias, y_pre=pre2,
                                                                           d_amax_g=amax, act=fp8lin.ACT_SWIGLU)))
            for name, fn in runs:
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                s.record()
                for _ in range(iters):
                    fn()
                e.record()
                torch.cuda.synchronize()
                t = s.elapsed_time(e) / iters
                line += f" | {name} {2.0 * M * N * K / t / 1e9:7.1f} TF {t * 1e3:7.1f} us"
        print(line, flush=True)


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


def stack(ctx, shapes, steps=40, warmup=8, only=None, graph=True):
    """ms per SGD step of the stack of FP8 linears (torch glue included): every tensor scaled just in time with
    separate activation kernels; activation and amax fused into the matmul epilogues; amax-history scaling with
    the FP8 bytes written by the epilogues."""
    from . import stack as S
    for layers, d, tokens in shapes:
        kw = dict(layers=layers, d=d, tokens=tokens)
        variants = (("just in time", lambda: S.Fp8Stack(ctx, **kw)),
                    ("fused epilogues", lambda: S.Fp8Stack(ctx, fused_activation=True, **kw)),
                    ("amax history", lambda: S.Fp8StackHistory(ctx, margin=1, **kw)))
        for name, make in variants:
            if only and only not in name:
                continue
            st = make()
            for i in range(warmup):
                st.step(i)
            torch.cuda.synchronize()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            for i in range(warmup, warmup + steps):
                r = st.step(i)
            e.record()
            torch.cuda.synchronize()
            ms = s.elapsed_time(e) / steps
            if not graph:
                print(f"stack {layers}x{d}x{tokens} {name:16s}: {ms:7.3f} ms/step  "
                      f"{st.flops_per_step() / ms / 1e9:7.1f} TFLOP/s | loss {float(r['loss'].item()):.5f}", flush=True)
                continue
            # the same step replayed from a CUDA graph: device time without the host's launch overhead
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                st.step(warmup + steps)
                with torch.cuda.graph(g, stream=side):
                    st.step(warmup + steps)
            torch.cuda.current_stream().wait_stream(side)
            g.replay()
            torch.cuda.synchronize()
            s.record()
            for _ in range(steps):
                g.replay()
            e.record()
            torch.cuda.synchronize()
            ms_graph = s.elapsed_time(e) / steps
            print(f"stack {layers}x{d}x{tokens} {name:16s}: {ms:7.3f} ms/step  {st.flops_per_step() / ms / 1e9:7.1f} TFLOP/s"
                  f" | from a CUDA graph {ms_graph:7.3f} ms/step  {st.flops_per_step() / ms_graph / 1e9:7.1f} TFLOP/s"
                  f" | loss {float(r['loss'].item()):.5f}", flush=True)
            del st, g


def mlp(ctx, shapes, iters=20, quiet=False):
    """Forward of a gated MLP (x -> SiLU(x Wg^T) * (x Wu^T) -> . Wd^T), every linear in FP8: (a) each linear quantises
    its input just in time and the gated unit is separate torch kernels; (b) the gate_up matmul's epilogue computes
    the gated unit and writes the down projection's FP8 input under a bias carried over from the previous call
    (amax-history scaling).  Weights are quantised once, outside the timed region, in both variants."""
    from . import inputs as I
    results = []
    say = (lambda *a, **k: None) if quiet else print
    for T, d, F in shapes:
        dev = dict(device="cuda")
        x = torch.randn(T, d, **dev).to(torch.bfloat16)
        wg, wu = (torch.randn(F, d, **dev) * 0.02).to(torch.bfloat16), (torch.randn(F, d, **dev) * 0.02).to(torch.bfloat16)
        wd = (torch.randn(d, F, **dev) * 0.02).to(torch.bfloat16)
        w_gu = torch.cat((wg, wu), 0).contiguous()           # unfused: gate rows then up rows
        w_il = I.interleave32(wg, wu).contiguous()           # fused: blocks of 32 gate rows, 32 up rows
        sc_f = torch.zeros(8, dtype=torch.float32, **dev)
        sc_i = torch.zeros(8, dtype=torch.int32, **dev)
        u8 = dict(dtype=torch.uint8, **dev)
        w_gu8, w_il8, wd8 = torch.empty((2 * F, d), **u8), torch.empty((2 * F, d), **u8), torch.empty((d, F), **u8)
        ctx.ptq_weights(w_gu, fp8lin.CONV_PAPER, w_gu8, None, sc_i[0:1], sc_f[0:1])
        ctx.ptq_weights(w_il, fp8lin.CONV_PAPER, w_il8, None, sc_i[1:2], sc_f[1:2])
        ctx.ptq_weights(wd, fp8lin.CONV_PAPER, wd8, None, sc_i[2:3], sc_f[2:3])
        x8, z8 = torch.empty((T, d), **u8), torch.empty((T, F), **u8)
        h = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)
        out = torch.empty((T, d), dtype=torch.bfloat16, **dev)

        def unfused():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd(x8, sc_i[3:4], w_gu8, sc_i[0:1], h)
            z = (torch.nn.functional.silu(h[:, :F].float()) * h[:, F:].float()).to(torch.bfloat16)
            ctx.cast_e4(z, None, d_amax_out=sc_f[4:5], d_bias_out=sc_i[4:5], y=z8)
            ctx.linear_fwd(z8, sc_i[4:5], wd8, sc_i[2:3], out)

        def fused():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd_q(x8, sc_i[3:4], w_il8, sc_i[1:2], z8, sc_i[5:6], d_amax_z=sc_f[5:6], act=fp8lin.ACT_SWIGLU)
            ctx.linear_fwd(z8, sc_i[5:6], wd8, sc_i[2:3], out)
            ctx.scaling_bias(sc_f[5:6], fp8lin.E4, fp8lin.CONV_PAPER, 1, sc_i[5:6])   # next call's bias, margin 1

        unfused()
        sc_i[5:6].copy_(sc_i[4:5] - 1)                       # history for the first fused call
        res = {}
        for name, fn in (("unfused", unfused), ("SwiGLU epilogue", fused)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            for _ in range(iters):
                fn()
            e.record()
            torch.cuda.synchronize()
            res[name] = s.elapsed_time(e) / iters
        flops = 2.0 * T * d * 3 * F
        say(f"mlp T={T} d={d} ffn={F} forward: " + " | ".join(f"{k} {v:7.3f} ms {flops / v / 1e9:7.1f} TFLOP/s" for k, v in res.items()),
            flush=True)
        results.append({"tokens": T, "d": d, "ffn": F, "pass": "fwd", "unfused_ms": res["unfused"],
                        "fused_ms": res["SwiGLU epilogue"], "fused_tflops": flops / res["SwiGLU epilogue"] / 1e9})
        if T < 256:
            continue
        # ---- forward + backward of the same block (training step without the optimiser) ----
        dy = (torch.randn(T, d, **dev) * 1e-3).to(torch.bfloat16)
        dy8, g8 = torch.empty((T, d), **u8), torch.empty((T, 2 * F), **u8)
        dz = torch.empty((T, F), dtype=torch.bfloat16, **dev)
        dx = torch.empty((T, d), dtype=torch.bfloat16, **dev)
        dw_gu = torch.empty((2 * F, d), dtype=torch.bfloat16, **dev)
        dw_d = torch.empty((d, F), dtype=torch.bfloat16, **dev)
        h_il = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)

        def unfused_step():
            unfused()
            ctx.cast_e5(dy, None, d_amax_out=sc_f[6:7], d_bias_out=sc_i[6:7], y=dy8)
            ctx.linear_dgrad(dy8, sc_i[6:7], wd8, None, sc_i[2:3], dz)
            ctx.linear_wgrad(dy8, None, sc_i[6:7], z8, None, sc_i[4:5], dw_d, T)
            a, u_ = h[:, :F].float(), h[:, F:].float()
            sg = torch.sigmoid(a)
            g = torch.cat(((dz.float() * u_ * (sg + a * sg * (1 - sg))), (dz.float() * a * sg)), 1).to(torch.bfloat16)
            ctx.cast_e5(g, None, d_amax_out=sc_f[7:8], d_bias_out=sc_i[7:8], y=g8)
            ctx.linear_dgrad(g8, sc_i[7:8], w_gu8, None, sc_i[0:1], dx)
            ctx.linear_wgrad(g8, None, sc_i[7:8], x8, None, sc_i[3:4], dw_gu, T)

        gb = torch.zeros(2, dtype=torch.int32, **dev)      # history bias of the gate/up gradient, and its next value
        ga = torch.zeros(1, dtype=torch.float32, **dev)

        def fused_step():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd_q(x8, sc_i[3:4], w_il8, sc_i[1:2], z8, sc_i[5:6], y_pre=h_il, d_amax_z=sc_f[5:6],
                             act=fp8lin.ACT_SWIGLU)
            ctx.linear_fwd(z8, sc_i[5:6], wd8, sc_i[2:3], out)
            ctx.cast_e5(dy, None, d_amax_out=sc_f[6:7], d_bias_out=sc_i[6:7], y=dy8)
            ctx.linear_dgrad_q(dy8, sc_i[6:7], wd8, None, sc_i[2:3], g8, gb[0:1], y_pre=h_il, d_amax_g=ga,
                               act=fp8lin.ACT_SWIGLU)
            ctx.linear_wgrad(dy8, None, sc_i[6:7], z8, None, sc_i[5:6], dw_d, T)
            ctx.linear_dgrad(g8, gb[0:1], w_il8, None, sc_i[1:2], dx)
            ctx.linear_wgrad(g8, None, gb[0:1], x8, None, sc_i[3:4], dw_gu, T)
            ctx.scaling_bias(sc_f[5:6], fp8lin.E4, fp8lin.CONV_PAPER, 1, sc_i[5:6])
            ctx.scaling_bias(ga, fp8lin.E5, fp8lin.CONV_PAPER, 1, gb[0:1])

        unfused_step()
        gb[0:1].copy_(sc_i[7:8] - 1)
        res = {}
        for name, fn in (("unfused", unfused_step), ("SwiGLU epilogues", fused_step)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            s.record()
            for _ in range(iters):
                fn()
            e.record()
            torch.cuda.synchronize()
            res[name] = s.elapsed_time(e) / iters
        flops *= 3
        say(f"mlp T={T} d={d} ffn={F} forward + backward: "
            + " | ".join(f"{k} {v:7.3f} ms {flops / v / 1e9:7.1f} TFLOP/s" for k, v in res.items()), flush=True)
        results.append({"tokens": T, "d": d, "ffn": F, "pass": "fwd+bwd", "unfused_ms": res["unfused"],
                        "fused_ms": res["SwiGLU epilogues"], "fused_tflops": flops / res["SwiGLU epilogues"] / 1e9})
    return results


def main(argv):
    opts = {"--only": None, "--steps": None, "--warmup": None}
    graph = "--no-graph" not in argv
    argv = [a for a in argv if a != "--no-graph"]
    for key in opts:
        if key in argv:
            i = argv.index(key)
            opts[key] = argv[i + 1]
            del argv[i:i + 2]
    if len(argv) < 2 or argv[0] not in ("gemm", "cast", "stack", "mlp"):
        print(__doc__)
        return 2
    shapes = [tuple(int(v) for v in a.split("x")) for a in argv[1:]]
    ctx = fp8lin.Context(0)
    if argv[0] == "stack":
        stack(ctx, shapes, steps=int(opts["--steps"] or 40), warmup=int(opts["--warmup"] or 8), only=opts["--only"],
              graph=graph)
    else:
        {"gemm": gemm, "cast": cast, "mlp": mlp}[argv[0]](ctx, shapes)
    flags = ctx.device_flags()
    if flags & fp8lin.FLAG_TIMEOUT:
        print("a device-side wait expired", file=sys.stderr)
        return 3
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
