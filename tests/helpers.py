"""Shared helpers for the GPU parity tests (marshalling and comparisons only)."""
import numpy as np
import torch

import oracle as O


def bits_of(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device) -> numpy uint16 bit patterns."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_from_bits(b: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(b).view(np.int16).copy()).view(torch.bfloat16).to(device)


def u8(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().cpu().numpy()


def assert_codes_equal(got: np.ndarray, want: np.ndarray, fmt: int):
    """Bit-exact FP8 bytes; NaN codes are compared by class."""
    table = O.decode_table(fmt)
    nan_w = np.isnan(table[want])
    nan_g = np.isnan(table[got])
    assert np.array_equal(nan_w, nan_g), "NaN positions differ"
    bad = (got != want) & ~nan_w
    if bad.any():
        idx = np.argwhere(bad)[:5]
        raise AssertionError(f"{bad.sum()} FP8 bytes differ, first at {idx.tolist()}: "
                             f"got {[hex(got[tuple(i)]) for i in idx]} want {[hex(want[tuple(i)]) for i in idx]}")


def bf16_ordinal(b: np.ndarray) -> np.ndarray:
    """Monotone integer key of bf16 bit patterns (sign-magnitude -> ordered)."""
    b = b.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def assert_gemm_close(got_f32: np.ndarray, ref: "O.GemmResult"):
    """FP32 result within 2^-14 * sum_k |a*b| of the exact value (plus half
    the smallest FP32 subnormal, below which no FP32 output can resolve)."""
    err = np.abs(got_f32.astype(np.float64) - ref.f64)
    tol = ref.abs_sum * 2.0 ** -14 + 2.0 ** -150
    bad = ~(err <= tol)
    if bad.any():
        i = np.argwhere(bad)[0]
        raise AssertionError(f"{bad.sum()} of {bad.size} outputs out of tolerance; first at {i.tolist()}: "
                             f"got {got_f32[tuple(i)]} want {ref.f64[tuple(i)]} tol {tol[tuple(i)]}")
    return float((err / np.maximum(ref.abs_sum, 1e-300)).max())


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def assert_bf16_within_one_ulp(got_bits: np.ndarray, ref: "O.GemmResult"):
    """bf16 output within one bf16 ulp of the oracle's rounded value.  Where the
    sum cancels, one bf16 ulp of the result is finer than the FP32 accumulation
    bar (2^-14 * sum_k |a*b|); there that bar, plus the half ulp of the output
    rounding itself, is the one that applies."""
    d = np.abs(bf16_ordinal(got_bits) - bf16_ordinal(ref.bf16))
    got = bf16_bits_to_f64(got_bits)
    half_ulp = np.abs(ref.f64) * 2.0 ** -8
    within_acc = np.abs(got - ref.f64) <= ref.abs_sum * 2.0 ** -14 + half_ulp + 2.0 ** -150
    bad = (d > 1) & ~within_acc
    if bad.any():
        i = np.argwhere(bad)[0]
        raise AssertionError(f"{bad.sum()} bf16 outputs differ by more than one ulp; first at {i.tolist()}: "
                             f"got {hex(got_bits[tuple(i)])} want {hex(ref.bf16[tuple(i)])}")
    return float((d > 1).mean())
