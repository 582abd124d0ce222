"""Seeded synthetic tensors shaped like the paper's GPT and Llama 2 linear layers.

This module holds no arithmetic of the method (no amax, bias, cast or matmul):
it only draws bf16 tensors, so that the CUDA path and the CPU oracle can be fed
the very same bits.  Values come from a counter-based generator -- element
``i`` of tensor ``tensor_id`` under ``seed`` is a pure function of
``(seed, tensor_id, i)`` -- so any slice can be regenerated on its own, on the
CPU or on the GPU.  (libm differences between devices can move a value by one
bf16 ulp; every comparison in this repository hands one generated tensor to
both sides, so that never matters.)

Model widths follow Table 1 of the paper (GPT 111M / 1.3B, Llama 2 7B / 70B)
and the four quantised linears per decoder layer follow Appendix E.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import torch

BASE_SEED = 230917224

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int -> the int64 two's-complement value with the same 64 bits."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    return (z >> k) & ((1 << (64 - k)) - 1)


def _splitmix64(z: torch.Tensor) -> torch.Tensor:
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _splitmix64_int(v: int) -> int:
    z = (v + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _stream_key(seed: int, tensor_id: int, salt: int = 0) -> int:
    return _splitmix64_int(_splitmix64_int(seed) ^ _splitmix64_int(tensor_id * 0x100000001B3 + salt))


def _normals(key: int, start: int, count: int, device) -> torch.Tensor:
    """Standard normals (float64) for flat indices [start, start+count)."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = _splitmix64(idx + _s64(key))
    u1 = (((h >> 40) & 0xFFFFFF).to(torch.float64) + 0.5) * (1.0 / (1 << 24))
    u2 = (((h >> 16) & 0xFFFFFF).to(torch.float64) + 0.5) * (1.0 / (1 << 24))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def outlier_columns(cols: int, frac: float, seed: int, tensor_id: int, device="cpu") -> torch.Tensor:
    """Boolean mask of the feature columns that carry outliers (fixed per tensor)."""
    if frac <= 0.0:
        return torch.zeros(cols, dtype=torch.bool, device=device)
    key = _stream_key(seed, tensor_id, salt=1)
    h = _splitmix64(torch.arange(cols, dtype=torch.int64, device=device) + _s64(key))
    u = ((h >> 40) & 0xFFFFFF).to(torch.float64) * (1.0 / (1 << 24))
    return u < frac


def uniform_scalar(seed: int, tensor_id: int, salt: int, lo: float, hi: float) -> float:
    """One uniform draw in [lo, hi) tied to (seed, tensor_id, salt)."""
    h = _splitmix64_int(_stream_key(seed, tensor_id, salt=1000 + salt))
    return lo + (hi - lo) * ((h >> 11) / float(1 << 53))


def normal_bf16(rows: int, cols: int, std: float, seed: int, tensor_id: int, device="cpu",
                outlier_frac: float = 0.0, outlier_scale: float = 1.0, log2_scale: float = 0.0,
                chunk_rows: int = 0) -> torch.Tensor:
    """bf16 [rows, cols] ~ N(0, std) * 2^log2_scale, with a fraction of the
    columns multiplied by ``outlier_scale``; rounding to bf16 is nearest-even."""
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    key = _stream_key(seed, tensor_id)
    mask = outlier_columns(cols, outlier_frac, seed, tensor_id, device)
    col_scale = torch.where(mask, torch.tensor(float(outlier_scale), dtype=torch.float64, device=device),
                            torch.tensor(1.0, dtype=torch.float64, device=device))
    col_scale = col_scale * (std * 2.0 ** log2_scale)
    if chunk_rows <= 0:
        chunk_rows = max(1, (1 << 23) // max(1, cols))
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        z = _normals(key, r0 * cols, (r1 - r0) * cols, device).view(r1 - r0, cols)
        out[r0:r1] = (z * col_scale).to(torch.float32).to(torch.bfloat16)
    return out


# ----------------------------------------------------------------------------
# workload definitions
# ----------------------------------------------------------------------------

@dataclass(frozen=True)
class Layer:
    name: str
    K: int  # in-features
    N: int  # out-features


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    layers: Tuple[Layer, ...]
    x_std: float = 1.0
    x_outlier_frac: float = 0.0
    x_outlier_scale: float = 1.0
    w_std: float = 0.02
    g_std: float = 1e-3
    g_log2_range: Tuple[float, float] = (0.0, 0.0)  # per-step log-uniform magnitude of dY
    backward: bool = True
    config_id: int = 0

    def flops(self, tokens: int = 0) -> float:
        t = tokens or self.tokens
        per = sum(2.0 * t * l.K * l.N for l in self.layers)
        return per * (3 if self.backward else 1)


WORKLOADS: Dict[str, Workload] = {
    # one layer at GPT-111M width
    "c1_single": Workload("c1_single", 256, (Layer("fc", 768, 768),), g_std=1e-3, config_id=1),
    # GPT 1.3B-width block
    "c2_gpt": Workload("c2_gpt", 4096,
                       (Layer("qkv", 2048, 6144), Layer("out", 2048, 2048),
                        Layer("ffn_up", 2048, 8192), Layer("ffn_down", 8192, 2048)),
                       x_outlier_frac=0.01, x_outlier_scale=50.0, g_std=1e-4,
                       g_log2_range=(-12.0, -4.0), config_id=2),
    # Llama 2 7B block
    "c3_llama7b": Workload("c3_llama7b", 8192,
                           (Layer("qkv", 4096, 12288), Layer("o", 4096, 4096),
                            Layer("gate_up", 4096, 22016), Layer("down", 11008, 4096)),
                           x_outlier_frac=0.005, x_outlier_scale=100.0, g_std=1e-5, config_id=3),
    # Llama 2 70B block, post-training quantisation, forward only
    "c4_llama70b_ptq": Workload("c4_llama70b_ptq", 2048,
                                (Layer("qkv", 8192, 10240), Layer("o", 8192, 8192),
                                 Layer("gate_up", 8192, 57344), Layer("down", 28672, 8192)),
                                x_outlier_frac=0.005, x_outlier_scale=100.0, w_std=0.015,
                                backward=False, config_id=4),
}

X_ID, W_ID, G_ID, TARGET_ID = 0, 1, 2, 3


def tensor_id(config_id: int, layer_index: int, which: int) -> int:
    return config_id * 1000 + layer_index * 10 + which


def layer_tensors(wl: Workload, layer_index: int, device="cpu", seed: int = BASE_SEED, step: int = 0,
                  tokens: int = 0, want=("x", "w", "g")):
    """bf16 X[T,K], W[N,K], dY[T,N] of one layer of a workload."""
    l = wl.layers[layer_index]
    T = tokens or wl.tokens
    out = {}
    if "x" in want:
        out["x"] = normal_bf16(T, l.K, wl.x_std, seed, tensor_id(wl.config_id, layer_index, X_ID), device,
                               wl.x_outlier_frac, wl.x_outlier_scale)
    if "w" in want:
        out["w"] = normal_bf16(l.N, l.K, wl.w_std, seed, tensor_id(wl.config_id, layer_index, W_ID), device)
    if "g" in want and wl.backward:
        lo, hi = wl.g_log2_range
        u = uniform_scalar(seed, tensor_id(wl.config_id, layer_index, G_ID), step, lo, hi) if hi > lo else 0.0
        out["g"] = normal_bf16(T, l.N, wl.g_std, seed + step, tensor_id(wl.config_id, layer_index, G_ID), device,
                               log2_scale=u)
    return out


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")


def interleave32(gate: torch.Tensor, up: torch.Tensor) -> torch.Tensor:
    """Rows of `gate` and `up` ([F, ...] each, F a multiple of 32) merged into [2F, ...] in blocks of 32 gate rows
    followed by their 32 up rows: the weight layout the SwiGLU epilogue expects (pure data movement)."""
    F = gate.shape[0]
    assert up.shape == gate.shape and F % 32 == 0
    rest = gate.shape[1:]
    return torch.stack((gate.reshape(F // 32, 32, *rest), up.reshape(F // 32, 32, *rest)), dim=1).reshape(2 * F, *rest)
