"""CPU-side checks of the C-ABI library: it loads, exports every symbol the
header declares, rejects bad arguments before touching a device, and its
host-side bias rule agrees with the oracle on every bf16 amax."""
import ctypes
import os
import re

import numpy as np
import torch

import oracle as O
from paper_2309_17224_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _lib():
    B.build()
    from paper_2309_17224_b200 import fp8lin
    return fp8lin


def test_library_exports_every_declared_symbol():
    fp8lin = _lib()
    import glob
    header = "".join(open(h).read() for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))))
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(fp8h?_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(fp8lin.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared but not exported"
    assert declared == set(fp8lin.SYMBOLS)


def test_status_strings():
    fp8lin = _lib()
    assert fp8lin.status_string(0) == "ok"
    assert len({fp8lin.status_string(i) for i in range(8)}) == 8


def test_null_arguments_are_rejected_without_a_device():
    fp8lin = _lib()
    lib = fp8lin.raw()
    assert lib.fp8_create(None, 0) == fp8lin.ERR_NULL
    assert lib.fp8_destroy(None) == fp8lin.ERR_NULL
    assert lib.fp8_amax(None, None, 0, 1, 1, 1, None, None) == fp8lin.ERR_NULL
    assert lib.fp8_scaling_bias(None, None, 0, 0, 0, None, None) == fp8lin.ERR_NULL
    assert lib.fp8_cast_e4(None, None, 0, 1, 1, 1, None, 0, 0, None, None, None, None, None) == fp8lin.ERR_NULL
    assert lib.fp8_linear_fwd(None, None, None, None, None, None, 0, None, 0, None, 1, 16, 1, 0, None) == fp8lin.ERR_NULL
    assert lib.fp8_scaling_bias_host(ctypes.c_float(1.0), 0, 0, 0, None) == fp8lin.ERR_NULL
    out = ctypes.c_int32()
    assert lib.fp8_scaling_bias_host(ctypes.c_float(1.0), 7, 0, 0, ctypes.byref(out)) == fp8lin.ERR_DTYPE


def test_host_bias_rule_matches_the_oracle_for_every_bf16_amax():
    fp8lin = _lib()
    bits = np.arange(0, 0x8000, dtype=np.uint32).astype(np.uint16)
    vals = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    for fmt, conv in ((O.E4, O.CONV_PAPER), (O.E4, O.CONV_NATIVE), (O.E5, O.CONV_PAPER), (O.E5, O.CONV_NATIVE)):
        for margin in (0, 3):
            for v in vals[::3]:
                assert fp8lin.scaling_bias_host(float(v), fmt, conv, margin) == O.scaling_bias(float(v), fmt, conv, margin)
    # float32 amax values that are not bf16 values (e.g. an amax taken from an FP32 output), subnormals included
    rng = np.random.default_rng(0)
    f32 = rng.integers(1, 0x7F800000, size=4000, dtype=np.uint32).view(np.float32)
    f32 = np.concatenate([f32, np.array([1e-45, 3e-42, 1.17e-38, 240.0, 240.00002, 448.0, 57344.0, 57344.004], np.float32)])
    for v in f32:
        for fmt, conv in ((O.E4, O.CONV_PAPER), (O.E4, O.CONV_NATIVE), (O.E5, O.CONV_PAPER)):
            assert fp8lin.scaling_bias_host(float(v), fmt, conv, 0) == O.scaling_bias(float(v), fmt, conv, 0), v
