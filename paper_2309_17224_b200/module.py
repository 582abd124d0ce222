"""``Fp8Linear``: a drop-in ``torch.nn.Linear`` whose three matmuls run in FP8.

The layer the paper describes (Section 2: Fig. 3b, Eq. 1-3 and Section 2.2 for
the backward pass; Section 3 for the two ways of choosing the scaling bias;
Section 3.1 for inference on weights quantised once), wired into autograd.
Everything numeric happens in the C-ABI library: this file allocates buffers,
keeps the per-tensor device scalars (amax and scaling bias of W, X and dY) and
marshals arguments.  The one exception is the gradient of the optional additive
bias vector, which the paper's layer does not have: it is ``dY.sum(0)`` in torch.

Scaling policies (``scaling=``):

``"amax"``      FP8-AMAX, just in time (Eq. 3): every tensor is quantised under
                the bias of its own current amax (two passes over the tensor).
``"predicted"`` FP8-AMAX in one pass: each tensor is cast under the bias its
                previous step left behind while its amax is taken; where Eq. 3
                gives another bias the cast is repeated.  Same bits as "amax".
``"constant"``  FP8-CSCALE (Section 3): the caller's constant biases
                (``constant_bias=(b_w, b_x, b_g)``), no amax at all.

``margin`` (Section 3.2) is subtracted from the gradient's bias.  In ``eval()``
mode the weight is quantised once and cached until ``train()`` is called again
or ``requantise()`` is asked for (post-training quantisation); activations of at
most 64 KB are then quantised inside the matmul's own launch.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import fp8lin

_W, _X, _G = 0, 1, 2
_default_ctx = {}


def default_context(device: int) -> "fp8lin.Context":
    """One library context per device, created on first use (it owns the split-contraction workspace)."""
    if device not in _default_ctx:
        _default_ctx[device] = fp8lin.Context(device)
    return _default_ctx[device]


def _out_dtype(dt):
    """The library writes bf16 or fp32: fp16 tensors get bf16 results."""
    return dt if dt in (torch.bfloat16, torch.float32) else torch.bfloat16


class _Fp8LinearFn(torch.autograd.Function):
    @staticmethod
    def forward(fn, x, weight, bias_vec, layer):
        lib = layer.ctx
        K, N = layer.in_features, layer.out_features
        x2 = x.reshape(-1, K)
        if not x2.is_contiguous():
            x2 = x2.contiguous()
        T = x2.shape[0]
        dev = x2.device
        x8 = torch.empty((T, K), dtype=torch.uint8, device=dev)
        y = torch.empty((T, N), dtype=layer.out_dtype or _out_dtype(x.dtype), device=dev)
        am, bi = layer.amax, layer.bias_words
        if layer.training and layer.scaling != "constant" and T > 128:
            # training: W and X are quantised together, all passes of both tensors in two launches (fp8_cast_group)
            w8 = torch.empty((N, K), dtype=torch.uint8, device=dev)
            lib.cast_group([(fp8lin.E4, weight.detach(), am[_W:_W + 1], bi[_W:_W + 1], w8),
                            (fp8lin.E4, x2, am[_X:_X + 1], bi[_X:_X + 1], x8)], conv=layer.conv,
                           predicted=layer.scaling == "predicted")
            lib.linear_fwd(x8, bi[_X:_X + 1], w8, bi[_W:_W + 1], y, bias_vec=bias_vec, conv=layer.conv)
            fn.layer, fn.x_shape, fn.has_bias = layer, x.shape, bias_vec is not None
            fn.save_for_backward(x8, w8, bi[:2].clone())
            return y.reshape(*x.shape[:-1], N)
        w8, w8_is_old = layer._quantised_weight(weight)
        # the inference calls may read the weight's bytes early: only once those were written by an earlier forward pass
        frozen = (not layer.training) and w8_is_old
        if frozen and layer.scaling != "constant" and T <= 128:
            # inference on a few rows: the activation is quantised by the matmul's own launch where it is small enough
            lib.linear_infer_cast(x2, am[_X:_X + 1], bi[_X:_X + 1], x8, w8, bi[_W:_W + 1], y, bias_vec=bias_vec,
                                  conv=layer.conv)
        else:
            layer._quantise(fp8lin.E4, x2, _X, x8, margin=0)
            run = lib.linear_infer if frozen else lib.linear_fwd
            run(x8, bi[_X:_X + 1], w8, bi[_W:_W + 1], y, bias_vec=bias_vec, conv=layer.conv)
        fn.layer = layer
        fn.x_shape = x.shape
        fn.has_bias = bias_vec is not None
        # X8 and W8 are cast once in the forward pass and used again by the backward matmuls (Section 2.2); their
        # biases are copied because the layer's words are rewritten by its next forward pass
        fn.save_for_backward(x8, w8, bi[:2].clone())
        return y.reshape(*x.shape[:-1], N)

    @staticmethod
    def backward(fn, dy):
        layer = fn.layer
        lib = layer.ctx
        K, N = layer.in_features, layer.out_features
        x8, w8, b_fwd = fn.saved_tensors
        T = x8.shape[0]
        dy2 = dy.reshape(T, N)
        if not dy2.is_contiguous():
            dy2 = dy2.contiguous()
        g8 = torch.empty((T, N), dtype=torch.uint8, device=dy2.device)
        layer._quantise(fp8lin.E5, dy2, _G, g8, margin=layer.margin)
        bg = layer.bias_words[_G:_G + 1]
        dx = dw = db = None
        if fn.needs_input_grad[0]:
            dx = torch.empty((T, K), dtype=_out_dtype(dy.dtype), device=dy2.device)
        if fn.needs_input_grad[1]:
            dw = torch.empty((N, K), dtype=_out_dtype(layer.weight.dtype), device=dy2.device)
        if dx is not None and dw is not None:
            # the two backward matmuls share dY8 and do not depend on each other (Section 2.2): one launch
            lib.linear_group([(fp8lin.MATMUL_DGRAD, g8, bg, w8, b_fwd[_W:_W + 1], dx),
                              (fp8lin.MATMUL_WGRAD, g8, bg, x8, b_fwd[_X:_X + 1], dw)], conv=layer.conv)
        elif dx is not None:
            lib.linear_dgrad(g8, bg, w8, None, b_fwd[_W:_W + 1], dx, conv=layer.conv)
        elif dw is not None:
            lib.linear_wgrad(g8, None, bg, x8, None, b_fwd[_X:_X + 1], dw, T, conv=layer.conv)
        if dx is not None:
            dx = dx.reshape(fn.x_shape)
        if dw is not None and dw.dtype != layer.weight.dtype:
            dw = dw.to(layer.weight.dtype)
        if fn.has_bias and fn.needs_input_grad[2]:
            db = dy2.sum(0, dtype=torch.float32).to(layer.bias.dtype)   # not part of the paper's layer
        return dx, dw, db, None


class Fp8Linear(torch.nn.Module):
    """``y = x W^T (+ b)`` with X, W quantised to E4 and dY to E5 under per-tensor power-of-two scaling biases.

    weight: [out_features, in_features], bf16 (default) or fp32 master weights (the cast reads either); inputs and
    output gradients bf16, fp16 or fp32; outputs and gradients bf16 or fp32 (fp16 is not an output type of the
    library).  ``in_features`` must be a multiple of 16 (rows of FP8 bytes are fetched in 16-byte units).
    After a backward pass ``amax`` and ``bias_words`` hold the three tensors' statistics of that step
    (order W, X, dY), on the device; nothing here synchronises with the host."""

    def __init__(self, in_features: int, out_features: int, bias: bool = False, device="cuda", dtype=torch.bfloat16,
                 scaling: str = "amax", margin: int = 0, conv: int = fp8lin.CONV_PAPER,
                 constant_bias: Optional[Sequence[int]] = None, out_dtype=None, ctx: Optional["fp8lin.Context"] = None):
        super().__init__()
        if scaling not in ("amax", "predicted", "constant"):
            raise ValueError("scaling must be 'amax', 'predicted' or 'constant'")
        if scaling == "constant" and (constant_bias is None or len(constant_bias) != 3):
            raise ValueError("scaling='constant' needs constant_bias=(b_w, b_x, b_g)")
        if in_features % 16:
            raise ValueError("in_features must be a multiple of 16")
        dev = torch.device(device)
        self.in_features, self.out_features = in_features, out_features
        self.scaling, self.margin, self.conv, self.out_dtype = scaling, int(margin), conv, out_dtype
        self.ctx = ctx if ctx is not None else default_context(dev.index or 0)
        self.weight = torch.nn.Parameter(torch.empty((out_features, in_features), device=dev, dtype=dtype))
        self.bias = torch.nn.Parameter(torch.zeros(out_features, device=dev, dtype=dtype)) if bias else None
        torch.nn.init.normal_(self.weight, std=0.02)
        self.register_buffer("amax", torch.zeros(3, dtype=torch.float32, device=dev), persistent=False)
        init = list(constant_bias) if scaling == "constant" else [0, 0, 0]
        self.register_buffer("bias_words", torch.tensor(init, dtype=torch.int32, device=dev), persistent=False)
        self._w8 = None            # FP8 bytes of the weight, kept while the module is in eval() mode
        self._w8_version = None

    # -- quantisation -----------------------------------------------------------------------------------------------
    def _quantise(self, fmt, t, which, out8, margin):
        c = self.ctx
        a, b = self.amax[which:which + 1], self.bias_words[which:which + 1]
        cast = c.cast_e4 if fmt == fp8lin.E4 else c.cast_e5
        if self.scaling == "constant":
            cast(t, b, conv=self.conv, y=out8)
        elif self.scaling == "predicted":
            c.cast_predicted(fmt, t, a, b, out8, conv=self.conv, margin=margin)
        else:
            cast(t, None, conv=self.conv, margin=margin, d_amax_out=a, d_bias_out=b, y=out8)

    def _quantised_weight(self, weight):
        if not self.training and self._w8 is not None and self._w8_version == weight._version:
            return self._w8, True
        w8 = torch.empty((self.out_features, self.in_features), dtype=torch.uint8, device=weight.device)
        w = weight.detach()
        if not self.training and self.scaling != "constant":
            # post-training quantisation (Section 3.1): amax, bias and bytes once
            self.ctx.ptq_weights(w, self.conv, w8, None, self.bias_words[_W:_W + 1], self.amax[_W:_W + 1])
        else:
            self._quantise(fp8lin.E4, w, _W, w8, margin=0)
        if not self.training:
            self._w8, self._w8_version = w8, weight._version
        return w8, False

    def requantise(self):
        """Forget the cached FP8 weight (eval mode): the next forward pass quantises the weight again."""
        self._w8 = self._w8_version = None

    def train(self, mode: bool = True):
        self.requantise()
        return super().train(mode)

    def forward(self, x):
        return _Fp8LinearFn.apply(x, self.weight, self.bias, self)

    def extra_repr(self):
        return (f"in_features={self.in_features}, out_features={self.out_features}, bias={self.bias is not None}, "
                f"scaling={self.scaling}, margin={self.margin}")
