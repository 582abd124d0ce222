"""A stack of FP8 linears trained with SGD: the dynamic-scaling stress workload.

24 x (d -> d) FP8 linears with GELU between them, MSE loss to a seeded target,
plain SGD on FP32 master weights.  Every step re-quantises every weight,
activation and gradient tensor with a fresh FP8-AMAX bias, and the input scale
drifts as 2^(8 sin(step / 20)) so that the biases have to move.

Only the linears belong to the paper's method (``fp8_cast_e4/e5``,
``fp8_linear_fwd/dgrad/wgrad``); the glue around them (GELU and its
derivative, the loss gradient, the SGD update) is FP32 arithmetic rounded to
bf16, run by the library's harness kernels (``fp8h_*``, include/fp8_harness.h)
so that a step launches no framework kernels beyond its input and its loss.
``gelu_bf16`` / ``gelu_grad_f32`` below are the same formulas in torch, kept
for comparisons.
"""
from __future__ import annotations

import math
from typing import Dict, List

import torch

from . import fp8lin as _lib
from . import inputs as I

CONFIG_ID = 5
fp8lin_E4, fp8lin_E5, CONV_PAPER = 0, 1, 0   # enum values of the C ABI (formats, paper convention)
ACT_GELU = 1


def step_input(x_base: torch.Tensor, step: int) -> torch.Tensor:
    """bf16(X_base * 2^(8 sin(step/20))), the product taken in float64."""
    scale = 2.0 ** (8.0 * math.sin(step / 20.0))
    return (x_base.to(torch.float64) * scale).to(torch.float32).to(torch.bfloat16)


def gelu_bf16(y: torch.Tensor) -> torch.Tensor:
    z = y.to(torch.float32)
    return (0.5 * z * (1.0 + torch.erf(z * (1.0 / math.sqrt(2.0))))).to(torch.bfloat16)


def gelu_grad_f32(y: torch.Tensor) -> torch.Tensor:
    z = y.to(torch.float32)
    cdf = 0.5 * (1.0 + torch.erf(z * (1.0 / math.sqrt(2.0))))
    pdf = torch.exp(-0.5 * z * z) * (1.0 / math.sqrt(2.0 * math.pi))
    return cdf + z * pdf


class Fp8Stack:
    def __init__(self, ctx, layers: int = 24, d: int = 1024, tokens: int = 4096, lr: float = 1e-3,
                 seed: int = I.BASE_SEED, device="cuda", w_std: float = 0.02, fused_activation: bool = False,
                 log_steps: int = 0):
        """fused_activation: GELU runs in the forward matmul's epilogue, which also emits the amax of the
        activated tensor, so the next layer's input is quantised in one pass (no amax pass, no GELU kernel).
        log_steps > 0: every step appends the (amax, bias) of all 3 x layers tensors to a device-side ring that
        holds the last `log_steps` steps (``fp8_bias_log_append``); see ``bias_records`` / ``write_bias_csv`` /
        ``bias_modes``."""
        self.ctx, self.L, self.d, self.T, self.lr = ctx, layers, d, tokens, lr
        self.fused = fused_activation
        dev = dict(device=device)
        self.w32 = [I.normal_bf16(d, d, w_std, seed, I.tensor_id(CONFIG_ID, l, I.W_ID), device).to(torch.float32)
                    for l in range(layers)]
        self.x_base = I.normal_bf16(tokens, d, 1.0, seed, I.tensor_id(CONFIG_ID, 0, I.X_ID), device)
        self.target = I.normal_bf16(tokens, d, 1.0, seed, I.tensor_id(CONFIG_ID, 0, I.TARGET_ID), device)
        u8 = dict(dtype=torch.uint8, **dev)
        self.x8 = [torch.empty((tokens, d), **u8) for _ in range(layers)]
        self.x8t = [torch.empty((d, tokens), **u8) for _ in range(layers)]
        self.w8 = [torch.empty((d, d), **u8) for _ in range(layers)]
        self.w8t = [torch.empty((d, d), **u8) for _ in range(layers)]
        self.y = [torch.empty((tokens, d), dtype=torch.bfloat16, **dev) for _ in range(layers)]
        self.act = torch.empty((tokens, d), dtype=torch.bfloat16, **dev) if fused_activation else None
        self.gact = torch.empty((tokens, d), dtype=torch.bfloat16, **dev) if fused_activation else None
        self.g8 = torch.empty((tokens, d), **u8)
        self.g8t = torch.empty((d, tokens), **u8)
        self.dx = torch.empty((tokens, d), dtype=torch.bfloat16, **dev)
        self.dw = torch.empty((d, d), dtype=torch.bfloat16, **dev)
        self.w16 = [w.to(torch.bfloat16) for w in self.w32]      # bf16(W32), rewritten by every SGD update
        self.h = [torch.empty((tokens, d), dtype=torch.bfloat16, **dev) for _ in range(2)]   # GELU outputs, in turn
        self.g = [torch.empty((tokens, d), dtype=torch.bfloat16, **dev) for _ in range(2)]   # gradients, in turn
        # per layer: amax / bias of W, X, dY
        self.amax = torch.zeros((layers, 3), dtype=torch.float32, **dev)
        self.bias = torch.zeros((layers, 3), dtype=torch.int32, **dev)
        # bias log: one record {step, tensor id = 3 * layer + (0 W, 1 X, 2 dY), amax, bias} per tensor and step
        self.log_ring = torch.zeros((log_steps * 3 * layers, 4), dtype=torch.int32, **dev) if log_steps > 0 else None
        self.log_head = torch.zeros(1, dtype=torch.int64, **dev)
        # layers whose tensors the current step keeps copies of (inputs and outputs of every library call), for
        # comparisons made outside this module; empty in normal use
        self.snap_layers = ()
        self.snap: Dict[int, Dict[str, torch.Tensor]] = {}

    def _keep(self, l: int, **tensors) -> None:
        if l in self.snap_layers:
            self.snap.setdefault(l, {}).update({k: v.clone() for k, v in tensors.items()})

    def flops_per_step(self) -> float:
        return 3.0 * 2.0 * self.T * self.d * self.d * self.L

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        c = self.ctx
        have_amax = False   # the previous matmul's epilogue already produced amax(x)
        for l in range(self.L):
            w16 = self.w16[l]
            c.cast_e4(w16, None, d_amax_out=self.amax[l, 0:1], d_bias_out=self.bias[l, 0:1], y=self.w8[l], y_t=self.w8t[l])
            if have_amax:
                c.scaling_bias(self.amax[l, 1:2], fp8lin_E4, CONV_PAPER, 0, self.bias[l, 1:2])
                c.cast_e4(x, self.bias[l, 1:2], y=self.x8[l], y_t=self.x8t[l])
            else:
                c.cast_e4(x, None, d_amax_out=self.amax[l, 1:2], d_bias_out=self.bias[l, 1:2], y=self.x8[l], y_t=self.x8t[l])
            if self.fused and l + 1 < self.L:
                c.linear_fwd_act(self.x8[l], self.bias[l, 1:2], self.w8[l], self.bias[l, 0:1], self.y[l], self.act,
                                 d_amax_act=self.amax[l + 1, 1:2])
                x, have_amax = self.act, True
            else:
                c.linear_fwd(self.x8[l], self.bias[l, 1:2], self.w8[l], self.bias[l, 0:1], self.y[l])
                self._keep(l, x=x, w=w16, x8=self.x8[l], w8=self.w8[l], y=self.y[l])
                have_amax = False
                if l + 1 < self.L:
                    x = self.h[l % 2]
                    _lib.harness_gelu(self.y[l], x)
        return self.y[self.L - 1]

    def backward_and_update(self) -> None:
        c = self.ctx
        g = self.g[0]
        _lib.harness_mse_grad(self.y[self.L - 1], self.target, 2.0 / (self.T * self.d), g)
        have_amax = False   # the previous input-gradient matmul already produced amax(g)
        for l in range(self.L - 1, -1, -1):
            if have_amax:
                c.scaling_bias(self.amax[l, 2:3], fp8lin_E5, CONV_PAPER, 0, self.bias[l, 2:3])
                c.cast_e5(g, self.bias[l, 2:3], y=self.g8, y_t=self.g8t)
            else:
                c.cast_e5(g, None, d_amax_out=self.amax[l, 2:3], d_bias_out=self.bias[l, 2:3], y=self.g8, y_t=self.g8t)
            if self.fused and l > 0:
                # dX * GELU'(Y[l-1]) and its amax come straight out of the matmul
                c.linear_dgrad_act(self.g8, self.bias[l, 2:3], None, self.w8t[l], self.bias[l, 0:1], self.y[l - 1], None,
                                   self.gact, d_amax_act=self.amax[l - 1, 2:3])
            else:
                c.linear_dgrad(self.g8, self.bias[l, 2:3], None, self.w8t[l], self.bias[l, 0:1], self.dx)
                self._keep(l, dx=self.dx)
            c.linear_wgrad(None, self.g8t, self.bias[l, 2:3], None, self.x8t[l], self.bias[l, 1:2], self.dw, self.T)
            self._keep(l, g=g, g8=self.g8, dw=self.dw, amax=self.amax[l], bias=self.bias[l])
            _lib.harness_sgd(self.w32[l], self.dw, self.lr, self.w16[l])
            if l > 0:
                if self.fused:
                    g, have_amax = self.gact, True
                else:
                    g = self.g[l % 2]
                    _lib.harness_gelu_backward(self.dx, self.y[l - 1], g)

    def step(self, step: int, snap_layers=()) -> Dict[str, object]:
        """One training step.  `snap_layers`: layers whose tensors (every input and output of the library calls of
        this step) are copied into `self.snap[layer]`."""
        self.snap_layers, self.snap = tuple(snap_layers), {}
        x = step_input(self.x_base, step)
        out = self.forward(x)
        loss = torch.mean((out.to(torch.float32) - self.target.to(torch.float32)) ** 2)
        self.backward_and_update()
        self._log(step, self.bias)
        return {"loss": loss, "bias": self.bias.clone(), "amax": self.amax.clone()}

    # -- bias log (Appendix G / Appendix I style statistics) ---------------------------------------------------
    def _log(self, step: int, bias_used: torch.Tensor) -> None:
        if self.log_ring is not None:
            self.ctx.bias_log_append(self.log_ring, self.log_head, step, 0, self.amax.view(-1),
                                     bias_used.contiguous().view(-1))

    def bias_records(self):
        """The records currently in the ring, oldest first, as a list of (step, layer, tensor, amax, bias) with
        tensor in {"W", "X", "dY"}.  Synchronises."""
        if self.log_ring is None:
            return []
        ring = self.log_ring.cpu()
        head = int(self.log_head.item())
        cap = ring.shape[0]
        order = range(head - min(head, cap), head)
        amax = ring[:, 2].contiguous().view(torch.float32)
        out = []
        for n in order:
            r = ring[n % cap]
            tid = int(r[1])
            out.append((int(r[0]), tid // 3, ("W", "X", "dY")[tid % 3], float(amax[n % cap]), int(r[3])))
        return out

    def write_bias_csv(self, path: str) -> int:
        """step,layer,tensor,amax,bias for every record in the ring; returns the number of rows written."""
        rows = self.bias_records()
        with open(path, "w") as fh:
            fh.write("step,layer,tensor,amax,bias\n")
            for step, layer, tensor, amax, bias in rows:
                fh.write(f"{step},{layer},{tensor},{amax!r},{bias}\n")
        return len(rows)

    def bias_modes(self, step_lo: int, step_hi: int) -> torch.Tensor:
        """[layers, 3, 2] int32: per tensor, the mode of its bias over the logged steps in [step_lo, step_hi] and how
        often it occurred (``fp8_bias_mode``)."""
        out = torch.zeros((self.L, 3, 2), dtype=torch.int32, device=self.log_ring.device)
        for l in range(self.L):
            for j in range(3):
                self.ctx.bias_mode(self.log_ring, self.log_head, 3 * l + j, step_lo, step_hi, out[l, j, 0:1], out[l, j, 1:2])
        return out


class Fp8StackHistory(Fp8Stack):
    """The same stack with amax-history scaling (Section 3) for activations and gradients: each of those
    tensors is quantised with the bias Eq. 3 gives for its amax at the PREVIOUS step, minus ``margin``, by the
    epilogue of the matmul that produces it (``fp8_linear_fwd_q`` / ``fp8_linear_dgrad_q``), so no activation or
    gradient is read back for an amax pass or a cast; the amax that comes out of the same launch feeds the next
    step's bias.  Weights keep the just-in-time bias (they are re-quantised after every update).  The first
    step, which has no history, runs the just-in-time path.  No transposed copies: the backward matmuls read the
    forward layouts."""

    def __init__(self, ctx, margin: int = 1, **kw):
        super().__init__(ctx, fused_activation=True, **kw)
        self.margin = margin
        self.pred = torch.zeros_like(self.bias)       # [:, 1] activations, [:, 2] gradients
        self.have_history = False
        self.g8b = torch.empty_like(self.g8)

    def _update_history(self) -> None:
        c = self.ctx
        for l in range(self.L):
            c.scaling_bias(self.amax[l, 1:2], fp8lin_E4, CONV_PAPER, self.margin, self.pred[l, 1:2])
            c.scaling_bias(self.amax[l, 2:3], fp8lin_E5, CONV_PAPER, self.margin, self.pred[l, 2:3])
        self.have_history = True

    def step(self, step: int, snap_layers=()) -> Dict[str, object]:
        if not self.have_history:
            rec = super().step(step)
            self._update_history()
            return rec
        self.snap_layers, self.snap = tuple(snap_layers), {}
        c, L, T = self.ctx, self.L, self.T
        x = step_input(self.x_base, step)
        # the input of the first layer is the one activation no matmul produces: one pass, predicted bias
        c.cast_e4(x, self.pred[0, 1:2], margin=self.margin, d_amax_out=self.amax[0, 1:2],
                  d_bias_out=self.bias[0, 1:2], y=self.x8[0])
        # all weights were updated by the step before: one grouped call quantises them (FP8-AMAX, just in time)
        w16s = self.w16
        c.cast_group([(fp8lin_E4, w16s[l], self.amax[l, 0:1], self.bias[l, 0:1], self.w8[l]) for l in range(L)])
        for l in range(L):
            w16 = w16s[l]
            if l + 1 < L:
                c.linear_fwd_q(self.x8[l], self.pred[l, 1:2], self.w8[l], self.bias[l, 0:1], self.x8[l + 1],
                               self.pred[l + 1, 1:2], y_pre=self.y[l], d_amax_z=self.amax[l + 1, 1:2], act=ACT_GELU)
            else:
                c.linear_fwd(self.x8[l], self.pred[l, 1:2], self.w8[l], self.bias[l, 0:1], self.y[l])
            self._keep(l, w=w16, x8=self.x8[l], w8=self.w8[l], y=self.y[l], bias_x=self.pred[l, 1:2],
                       bias_w=self.bias[l, 0:1], **({"x8_next": self.x8[l + 1], "bias_next": self.pred[l + 1, 1:2],
                                                     "amax_next": self.amax[l + 1, 1:2]} if l + 1 < L else {}))
        loss = torch.mean((self.y[L - 1].to(torch.float32) - self.target.to(torch.float32)) ** 2)
        g = self.g[0]
        _lib.harness_mse_grad(self.y[L - 1], self.target, 2.0 / (T * self.d), g)
        bufs = (self.g8, self.g8b)
        c.cast_e5(g, self.pred[L - 1, 2:3], margin=self.margin, d_amax_out=self.amax[L - 1, 2:3],
                  d_bias_out=self.bias[L - 1, 2:3], y=bufs[(L - 1) % 2])
        for l in range(L - 1, -1, -1):
            cur, nxt = bufs[l % 2], bufs[(l + 1) % 2]
            if l > 0:
                c.linear_dgrad_q(cur, self.pred[l, 2:3], self.w8[l], None, self.bias[l, 0:1], nxt, self.pred[l - 1, 2:3],
                                 y_pre=self.y[l - 1], d_amax_g=self.amax[l - 1, 2:3], act=ACT_GELU)
            c.linear_wgrad(cur, None, self.pred[l, 2:3], self.x8[l], None, self.pred[l, 1:2], self.dw, T)
            self._keep(l, g8=cur, bias_g=self.pred[l, 2:3], dw=self.dw,
                       **({"g8_next": nxt, "bias_g_next": self.pred[l - 1, 2:3], "y_below": self.y[l - 1]} if l > 0 else {}))
            _lib.harness_sgd(self.w32[l], self.dw, self.lr, self.w16[l])
        used = self.bias.clone()
        used[:, 1:3] = self.pred[:, 1:3]
        rec = {"loss": loss, "bias": used, "amax": self.amax.clone()}
        self._log(step, used)
        self._update_history()
        return rec
