"""The constants of the GELU epilogue (CPU only): the script beside the kernel re-derives the polynomial of
`normal_lower_tail`, the kernel source must carry exactly those coefficients, and the float32 replay of the kernel's
arithmetic over every finite bf16 input must stay within one bf16 ulp of GELU from float64 erfc."""
import importlib.util
import pathlib
import re

CSRC = pathlib.Path(__file__).resolve().parents[1] / "paper_2309_17224_b200" / "csrc"


def _script():
    spec = importlib.util.spec_from_file_location("fit_normal_tail", CSRC / "fit_normal_tail.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_kernel_coefficients_are_the_fitted_ones_and_accurate_enough():
    fit = _script()
    coef, rel = fit.fit()
    assert rel < 5e-6
    src = (CSRC / "gemm.cu").read_text()
    body = src[src.index("float normal_lower_tail("):]
    body = body[:body.index("ex2.approx")]
    in_kernel = [float(m) for m in re.findall(r"(-?\d+\.\d+)f \* kTwoM32", body)]
    assert len(in_kernel) == len(coef) == 8
    for k, c in zip(in_kernel, reversed(coef)):          # Horner order in the kernel: highest power first
        assert abs(k - c) <= 1e-9 * max(1.0, abs(c)), (k, c)
    dmax, frac, grel = fit.check(in_kernel[::-1])
    assert dmax <= 1 and frac < 0.005 and grel < 2e-4
