"""GPU parity of ``Fp8Linear`` (the autograd wrapper around the C-ABI calls) against the CPU oracle.

The module only marshals arguments, so what is checked is the wiring: which tensor is cast in which format under
which bias, which buffers the backward matmuls reuse (Section 2.2), the margin on the gradient (Section 3.2), constant
biases (FP8-CSCALE, Section 3) and the cached weight of inference (Section 3.1).
"""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_bf16_within_one_ulp, assert_gemm_close, bits_of
from paper_2309_17224_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def M():
    from paper_2309_17224_b200 import module
    return module


def _tensors(T, K, N, seed):
    x = I.normal_bf16(T, K, 1.0, seed, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0)
    w = I.normal_bf16(N, K, 0.02, seed, 2, "cuda")
    g = I.normal_bf16(T, N, 1e-3, seed, 3, "cuda")
    return x, w, g


def _oracle_step(x, w, g, conv, margin, bias_vec=None):
    ax, bx, x8 = O.quantise(bits_of(x), O.E4, conv)
    aw, bw, w8 = O.quantise(bits_of(w), O.E4, conv)
    ag, bg, g8 = O.quantise(bits_of(g), O.E5, conv, margin)
    sx, sw, sg = bx + O.delta(O.E4, conv), bw + O.delta(O.E4, conv), bg + O.delta(O.E5, conv)
    y = O.linear_fwd(x8, sx, w8, sw, bias_vec=bias_vec)
    dx = O.linear_dgrad(g8, sg, w8, sw)
    dw = O.linear_wgrad(g8, sg, x8, sx)
    return (aw, ax, ag), (bw, bx, bg), y, dx, dw


@pytest.mark.parametrize("scaling", ["amax", "predicted"])
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_training_step_matches_the_oracle(M, scaling, conv):
    T, K, N = 400, 272, 528
    x, w, g = _tensors(T, K, N, 71)
    margin = 2
    layer = M.Fp8Linear(K, N, bias=True, scaling=scaling, margin=margin, conv=conv)
    bv = (torch.randn(N, device="cuda") * 0.1).to(torch.bfloat16)
    with torch.no_grad():
        layer.weight.copy_(w)
        layer.bias.copy_(bv)
    amaxes, biases, y_ref, dx_ref, dw_ref = _oracle_step(x, w, g, conv, margin, bias_vec=bv.double().cpu().numpy())
    for rnd in range(2):   # the second round starts from the first one's biases (what "predicted" guesses with)
        xin = x.view(4, 100, K).clone().requires_grad_(True)
        layer.zero_grad()
        y = layer(xin)
        assert y.shape == (4, 100, N) and y.dtype == torch.bfloat16
        y.backward(g.view(4, 100, N))
        assert_bf16_within_one_ulp(bits_of(y.detach().reshape(T, N)), y_ref)
        assert_bf16_within_one_ulp(bits_of(xin.grad.reshape(T, K)), dx_ref)
        assert_bf16_within_one_ulp(bits_of(layer.weight.grad), dw_ref)
        assert [float(a) for a in layer.amax.tolist()] == list(amaxes)
        assert layer.bias_words.tolist() == list(biases)
        torch.testing.assert_close(layer.bias.grad.float(), g.float().sum(0), rtol=1e-2, atol=1e-6)
    assert layer.ctx.device_flags(clear=True) & 8 == 0


def test_fp32_master_weights_and_fp32_results(M):
    T, K, N = 144, 1040, 304
    x, w, g = _tensors(T, K, N, 73)
    layer = M.Fp8Linear(K, N, dtype=torch.float32, out_dtype=torch.float32)
    with torch.no_grad():
        layer.weight.copy_(w.float())
    _, _, y_ref, dx_ref, dw_ref = _oracle_step(x, w, g, O.CONV_PAPER, 0)
    xin = x.float().requires_grad_(True)      # fp32 activations holding bf16 values: the cast reads them exactly
    y = layer(xin)
    y.backward(g.float())
    assert y.dtype == torch.float32 and layer.weight.grad.dtype == torch.float32 and xin.grad.dtype == torch.float32
    assert_gemm_close(y.detach().cpu().numpy(), y_ref)
    assert_gemm_close(xin.grad.cpu().numpy(), dx_ref)
    assert_gemm_close(layer.weight.grad.cpu().numpy(), dw_ref)


def test_constant_biases_are_fp8_cscale(M):
    T, K, N = 256, 768, 768
    x, w, g = _tensors(T, K, N, 79)
    const = (4, 2, 14)           # W, X, dY; the activation bias clips the outlier columns (the flag must say so)
    layer = M.Fp8Linear(K, N, scaling="constant", constant_bias=const)
    with torch.no_grad():
        layer.weight.copy_(w)
    x8, w8, g8 = (O.cast(bits_of(t), b + O.delta(k, O.CONV_PAPER), O.native_format(k))
                  for t, b, k in ((x, const[1], O.E4), (w, const[0], O.E4), (g, const[2], O.E5)))
    sx, sw, sg = const[1] + 1, const[0] + 1, const[2]
    xin = x.clone().requires_grad_(True)
    y = layer(xin)
    y.backward(g)
    assert_bf16_within_one_ulp(bits_of(y.detach()), O.linear_fwd(x8, sx, w8, sw))
    assert_bf16_within_one_ulp(bits_of(xin.grad), O.linear_dgrad(g8, sg, w8, sw))
    assert_bf16_within_one_ulp(bits_of(layer.weight.grad), O.linear_wgrad(g8, sg, x8, sx))
    assert layer.bias_words.tolist() == list(const)
    assert layer.ctx.device_flags(clear=True) & 4      # saturation reported, as for any clipping cast


@pytest.mark.parametrize("T", [1, 4, 64, 300])
def test_inference_keeps_the_weight_quantised_once(M, T):
    K, N = 2048, 784
    x, w, _ = _tensors(T, K, N, 83)
    layer = M.Fp8Linear(K, N)
    with torch.no_grad():
        layer.weight.copy_(w)
    layer.eval()
    _, bx, x8 = O.quantise(bits_of(x), O.E4)
    _, bw, w8 = O.quantise(bits_of(w), O.E4)
    ref = O.linear_fwd(x8, bx + 1, w8, bw + 1)
    with torch.no_grad():
        y1 = layer(x)            # quantises the weight (fp8_ptq_weights) and multiplies
        cached = layer._w8
        y2 = layer(x)            # from here on the cached bytes; few rows: activation quantised inside the matmul launch
        y3 = layer(x)
    assert layer._w8 is cached and np.array_equal(cached.cpu().numpy(), w8)
    for y in (y1, y2, y3):
        assert_bf16_within_one_ulp(bits_of(y), ref)
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16)) and torch.equal(y2.view(torch.int16), y3.view(torch.int16))
    assert layer.bias_words.tolist()[:2] == [bw, bx]
    # a weight update invalidates the cache; train() drops it
    with torch.no_grad():
        layer.weight.mul_(2.0)
        y4 = layer(x)
    assert layer._w8 is not cached
    assert_bf16_within_one_ulp(bits_of(y4), O.linear_fwd(x8, bx + 1, w8, bw))   # W doubled: its bias drops by one
    layer.train()
    assert layer._w8 is None
    assert layer.ctx.device_flags(clear=True) & 8 == 0


def test_a_two_layer_model_trains_with_an_optimizer(M):
    """Wiring check with torch's own machinery: two FP8 linears (FP32 master weights) and a GELU under Adam reduce a
    regression loss whose gradients are of the order of 1e-6 (what the E5 scaling bias is there for)."""
    torch.manual_seed(0)
    kw = dict(bias=True, scaling="predicted", dtype=torch.float32, out_dtype=torch.bfloat16)
    model = torch.nn.Sequential(M.Fp8Linear(256, 512, **kw), torch.nn.GELU(), M.Fp8Linear(512, 256, **kw))
    x = torch.randn(1024, 256, device="cuda").to(torch.bfloat16)
    target = torch.randn(1024, 256, device="cuda").to(torch.bfloat16) * 0.1
    opt = torch.optim.Adam(model.parameters(), lr=2e-3)
    losses = []
    for _ in range(40):
        opt.zero_grad()
        loss = torch.nn.functional.mse_loss(model(x).float(), target.float())
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    assert all(np.isfinite(losses))
    assert losses[-1] < 0.7 * losses[0], losses
