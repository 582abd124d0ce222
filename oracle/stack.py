"""CPU mirror of the 24-layer FP8 stress stack -- TEST INFRASTRUCTURE ONLY.

Same recipe as the GPU harness, written on the oracle's own functions: every
linear is oracle.quantise + the float64 matmul definitions; the glue (GELU,
its derivative, the MSE gradient, SGD) is float64 arithmetic rounded to
float32 and then to bf16, which is what "FP32 arithmetic rounded to bf16"
means up to the last bf16 ulp.  Inputs are the seeded tensors only.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf, erfc

import oracle as O


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    u = x.astype(np.float32).view(np.uint32).astype(np.uint64)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return np.where(nan, (u >> 16) | 0x40, rounded).astype(np.uint16)


def step_input_bits(x_base_bits: np.ndarray, step: int) -> np.ndarray:
    return f64_to_bf16(bf16_to_f64(x_base_bits) * 2.0 ** (8.0 * math.sin(step / 20.0)))


def gelu_bits(y_bits: np.ndarray) -> np.ndarray:
    """GELU(z) = z/2 * (1 + erf(z / sqrt 2)), written with erfc so that the far negative tail keeps its
    relative accuracy (1 + erf cancels there)."""
    z = bf16_to_f64(y_bits)
    return f64_to_bf16(0.5 * z * erfc(-z / math.sqrt(2.0)))


def gelu_grad(y_bits: np.ndarray) -> np.ndarray:
    z = bf16_to_f64(y_bits)
    return 0.5 * (1.0 + erf(z / math.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def _blocks32(two_f: int):
    """Column indices of the gate and of the up halves in the block layout [32 gate, 32 up, 32 gate, ...]."""
    assert two_f % 64 == 0
    j = np.arange(two_f // 2)
    gate = (j // 32) * 64 + j % 32
    return gate, gate + 32


def silu(a: np.ndarray) -> np.ndarray:
    """SiLU(a) = a * sigma(a); written per sign so that exp never overflows and the negative tail keeps its
    relative accuracy."""
    e = np.exp(-np.abs(a))
    return np.where(a > 0, a / (1.0 + e), a * e / (1.0 + e))


def swiglu_bits(y_pre_bits: np.ndarray) -> np.ndarray:
    """z[:, j] = bf16(SiLU(gate_j) * up_j) from the bf16 pre-activations [T, 2F] in the 32-block layout."""
    y = bf16_to_f64(y_pre_bits)
    gi, ui = _blocks32(y.shape[1])
    return f64_to_bf16(silu(y[:, gi]) * y[:, ui])


def swiglu_backward(dz: np.ndarray, y_pre_bits: np.ndarray) -> np.ndarray:
    """Gradients of the gate / up pre-activations, float64, in the 32-block layout:
    d_gate = dz * up * SiLU'(gate), d_up = dz * SiLU(gate), SiLU'(a) = s + a s (1 - s), s = sigma(a)."""
    y = bf16_to_f64(y_pre_bits)
    gi, ui = _blocks32(y.shape[1])
    a, u = y[:, gi], y[:, ui]
    e = np.exp(-np.abs(a))
    s = np.where(a > 0, 1.0 / (1.0 + e), e / (1.0 + e))
    out = np.empty_like(y)
    out[:, gi] = dz * u * (s + a * s * (1.0 - s))
    out[:, ui] = dz * silu(a)
    return out


class OracleStack:
    def __init__(self, w_bits, x_base_bits, target_bits, lr=1e-3, history=False, margin=0):
        """history: quantise every activation and gradient with the bias of Eq. 3 for that tensor's amax at the
        previous step, minus `margin` (the amax-history remedy of Section 3); weights, and every tensor at the
        first step, take the just-in-time bias."""
        self.w32 = [bf16_to_f64(w).astype(np.float32) for w in w_bits]
        self.x_base, self.target = x_base_bits, bf16_to_f64(target_bits)
        self.L = len(w_bits)
        self.lr = lr
        self.history, self.margin = history, margin
        self.prev_amax = None

    def _quantise(self, bits, kind, l, j):
        """(amax, bias used, bytes) of tensor j (1: activation, 2: gradient) of layer l."""
        if not self.history or self.prev_amax is None:
            return O.quantise(bits, kind)
        a = O.amax(bits)
        b = O.scaling_bias(float(self.prev_amax[l, j]), kind, O.CONV_PAPER, self.margin)
        return a, b, O.cast(bits, b + O.delta(kind, O.CONV_PAPER), O.native_format(kind))

    def step(self, step: int):
        """One training step.  Returns a record of every tensor a linear saw."""
        L = self.L
        T, d = self.x_base.shape
        rec = {"x": [], "w": [], "x8": [], "w8": [], "y": [], "g": [None] * L, "g8": [None] * L, "dx": [None] * L,
               "dw": [None] * L, "bias": np.zeros((L, 3), dtype=np.int64), "amax": np.zeros((L, 3))}
        x = step_input_bits(self.x_base, step)
        for l in range(L):
            w = f64_to_bf16(self.w32[l].astype(np.float64))
            aw, bw, w8 = O.quantise(w, O.E4)
            ax, bx, x8 = self._quantise(x, O.E4, l, 1)
            y = O.linear_fwd_np(x8, bx + 1, w8, bw + 1)
            rec["x"].append(x); rec["w"].append(w); rec["x8"].append(x8); rec["w8"].append(w8); rec["y"].append(y)
            rec["bias"][l, 0], rec["bias"][l, 1] = bw, bx
            rec["amax"][l, 0], rec["amax"][l, 1] = aw, ax
            if l + 1 < L:
                x = gelu_bits(y.bf16)
        out = bf16_to_f64(rec["y"][-1].bf16)
        rec["loss"] = float(np.mean((out - self.target) ** 2))
        g = f64_to_bf16((out - self.target) * (2.0 / (T * d)))
        for l in range(L - 1, -1, -1):
            ag, bg, g8 = self._quantise(g, O.E5, l, 2)
            bw, bx = int(rec["bias"][l, 0]), int(rec["bias"][l, 1])
            dx = O.linear_dgrad_np(g8, bg, rec["w8"][l], bw + 1)
            dw = O.linear_wgrad_np(g8, bg, rec["x8"][l], bx + 1)
            rec["g"][l], rec["g8"][l], rec["dx"][l], rec["dw"][l] = g, g8, dx, dw
            rec["bias"][l, 2], rec["amax"][l, 2] = bg, ag
            self.w32[l] = (self.w32[l].astype(np.float64) - self.lr * bf16_to_f64(dw.bf16)).astype(np.float32)
            if l > 0:
                g = f64_to_bf16(bf16_to_f64(dx.bf16) * gelu_grad(rec["y"][l - 1].bf16))
        self.prev_amax = rec["amax"].copy()
        return rec
