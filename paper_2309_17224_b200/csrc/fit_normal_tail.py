"""Derives and checks the polynomial behind `normal_lower_tail` in gemm.cu (the GELU epilogues).

    Phi(-|x|) = erfcx(z) / 2 * exp(-z^2),   z = |x| / sqrt 2,   erfcx(z) / 2 = t * Q(t),   t = 1 / (1 + z / 2)

Q is a degree-7 polynomial: a Chebyshev least-squares fit of erfcx(z) / (2 t) over t in (0, 1], i.e. all z >= 0.
The script prints Q's coefficients (monomial basis, float32) and then replays the kernel's arithmetic in float32
for EVERY finite bf16 input, against float64 erfc: the bf16-rounded GELU may differ from the correctly rounded one by
at most one bf16 ulp, and GELU' must stay within 2e-4 relative.  Run it after touching the coefficients:

    python paper_2309_17224_b200/csrc/fit_normal_tail.py

Needs numpy and scipy only; nothing imports this file.
"""
import math

import numpy as np
from numpy.polynomial import chebyshev as C
from numpy.polynomial import polynomial as P
from scipy.special import erfc, erfcx

DEGREE = 7
f32 = np.float32


def fit():
    t = (np.cos(np.pi * (np.arange(4000) + 0.5) / 4000) + 1) / 2      # Chebyshev nodes on (0, 1)
    z = 2 / t - 2
    target = 0.5 * erfcx(z) / t
    cheb = C.chebfit(2 * t - 1, target, DEGREE)
    rel = np.max(np.abs(C.chebval(2 * t - 1, cheb) / target - 1))
    mono = P.Polynomial(C.cheb2poly(cheb))(P.Polynomial([-1, 2])).coef   # substitute u = 2t - 1
    return [float(f32(c)) for c in mono], rel


def bf16_round(x):
    u = x.astype(np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def ordinal(b):
    b = b.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def check(coef):
    bits = np.arange(65536, dtype=np.uint32)
    x = (bits << 16).view(np.float32)
    x = x[np.isfinite(x)]
    a = np.abs(x)
    t = f32(1) / (a * f32(0.35355339059327373) + f32(1))
    q = np.full_like(t, f32(coef[-1]) * f32(2.0 ** -32))
    for k in range(DEGREE - 1, -1, -1):
        q = q * t + f32(coef[k]) * f32(2.0 ** -32)
    with np.errstate(over="ignore", under="ignore"):
        arg = ((x * x) * f32(-0.7213475204444817) + f32(32)).astype(f32)
        e = np.exp2(arg.astype(np.float64)).astype(f32)
        e = np.where(np.abs(e) < 2.0 ** -126, f32(0), e)              # the hardware exponential flushes to zero
    lower = (t * q * e).astype(f32)
    gelu = (np.maximum(x, f32(0)) - a * lower).astype(f32)
    x64 = x.astype(np.float64)
    exact = 0.5 * x64 * erfc(-x64 / math.sqrt(2))
    d = np.abs(ordinal(bf16_round(gelu)) - ordinal(bf16_round(exact.astype(np.float32))))
    cdf = np.where(x > 0, f32(1) - lower, lower).astype(f32)
    grad = (cdf + x * f32(0.3989422804014327 * 2.0 ** -32) * e).astype(f32)
    gexact = 0.5 * erfc(-x64 / math.sqrt(2)) + x64 * np.exp(-0.5 * x64 * x64) / math.sqrt(2 * math.pi)
    ok = np.abs(gexact) > 1e-30
    grel = (np.abs(grad - gexact) / np.maximum(np.abs(gexact), 1e-300))[ok].max()
    return int(d.max()), float((d > 0).mean()), float(grel)


if __name__ == "__main__":
    coef, rel = fit()
    print("Q(t) coefficients, t^0 .. t^%d:" % DEGREE)
    for c in coef:
        print("   %.9g" % c)
    print("fit: max relative error over z >= 0: %.2e" % rel)
    dmax, frac, grel = check(coef)
    print("GELU over all finite bf16 inputs: max distance %d bf16 ulp, %.2f %% of inputs differ" % (dmax, 100 * frac))
    print("GELU' over all finite bf16 inputs: max relative error %.2e" % grel)
    assert dmax <= 1 and grel < 2e-4
