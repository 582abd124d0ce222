"""B200-native FP8 linear layer with dynamically updated per-tensor scaling bias.

``paper_2309_17224_b200.fp8lin`` is the Python face of the C-ABI library
(``libfp8lin.so``, declared in ``include/fp8lin.h``); importing it fails loudly
when the library has not been built.  ``paper_2309_17224_b200.module`` wraps the
calls of one layer into ``Fp8Linear``, a ``torch.nn.Module`` with autograd.  ``paper_2309_17224_b200.inputs`` draws the
seeded synthetic tensors used by the tests and the benchmark.
"""
__all__ = ["fp8lin", "inputs", "build", "module"]
