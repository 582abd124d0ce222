"""Pins for the oracle's mirror of the stress stack (CPU only): its bf16
helpers and GELU against torch's float64 routines, and its backward pass
against float64 autograd of the same network without quantisation."""
import math

import numpy as np
import torch

import oracle as O
from oracle import stack as S


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _ord(b):
    b = b.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def test_bf16_helpers_match_torch():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(1000, 7, generator=g, dtype=torch.float64) * 100
    assert np.array_equal(S.f64_to_bf16(x.numpy()), _bits(x.to(torch.float32).to(torch.bfloat16)))
    b = _bits(x.to(torch.bfloat16))
    assert np.array_equal(S.bf16_to_f64(b), x.to(torch.bfloat16).to(torch.float64).numpy())


def test_step_input_drift():
    base = _bits(torch.tensor([[1.0, -3.0, 0.5]], dtype=torch.bfloat16))
    assert np.array_equal(S.step_input_bits(base, 0), base)
    # step 10 pi: sin = 0 again up to rounding of pi; step = 20*asin(0.5) gives 2^4
    s = 2.0 ** (8.0 * math.sin(7 / 20.0))
    want = _bits((torch.tensor([[1.0, -3.0, 0.5]], dtype=torch.float64) * s).to(torch.float32).to(torch.bfloat16))
    assert np.array_equal(S.step_input_bits(base, 7), want)


def test_gelu_and_its_derivative_against_torch_float64():
    y = (torch.linspace(-6, 6, 4001, dtype=torch.float64)).to(torch.bfloat16)
    yb = _bits(y.view(1, -1))
    ref = torch.nn.functional.gelu(y.to(torch.float64)).to(torch.float32).to(torch.bfloat16)
    assert np.abs(_ord(S.gelu_bits(yb)) - _ord(_bits(ref.view(1, -1)))).max() <= 1
    z = y.to(torch.float64).clone().requires_grad_(True)
    torch.nn.functional.gelu(z).sum().backward()
    np.testing.assert_allclose(S.gelu_grad(yb)[0], z.grad.numpy(), rtol=1e-12, atol=1e-15)


def test_stack_backward_is_the_gradient_of_its_forward():
    """Three small layers: the oracle's dW (FP8 path) must point along the
    float64 autograd gradient of the unquantised network, and one SGD step
    must lower the loss it reports."""
    rng = np.random.default_rng(5)
    L, T, d = 3, 128, 64
    w = [(torch.from_numpy(rng.standard_normal((d, d))) * 0.15).to(torch.bfloat16) for _ in range(L)]
    x = torch.from_numpy(rng.standard_normal((T, d))).to(torch.bfloat16)
    tgt = torch.from_numpy(rng.standard_normal((T, d))).to(torch.bfloat16)
    st = S.OracleStack([_bits(t) for t in w], _bits(x), _bits(tgt), lr=0.5)
    rec = st.step(0)
    ws = [t.to(torch.float64).clone().requires_grad_(True) for t in w]
    h = x.to(torch.float64)
    for l in range(L):
        h = h @ ws[l].T
        if l + 1 < L:
            h = torch.nn.functional.gelu(h)
    loss = torch.mean((h - tgt.to(torch.float64)) ** 2)
    loss.backward()
    assert abs(rec["loss"] - float(loss)) < 0.05 * float(loss)
    for l in range(L):
        mine = S.bf16_to_f64(rec["dw"][l].bf16).ravel()
        ref = ws[l].grad.numpy().ravel()
        cos = mine @ ref / (np.linalg.norm(mine) * np.linalg.norm(ref))
        assert cos > 0.98, (l, cos)
        assert 0.8 < np.linalg.norm(mine) / np.linalg.norm(ref) < 1.25
    assert st.step(0)["loss"] < rec["loss"]


def test_history_mode_uses_the_previous_steps_amax():
    """Amax-history scaling: step 0 is the just-in-time step; from step 1 on every activation / gradient bias
    is Eq. 3 on the previous step's amax minus the margin, the bytes are the cast under that bias (clipping
    where the tensor outgrew it), and weights keep their own just-in-time bias."""
    rng = np.random.default_rng(9)
    L, T, d, margin = 2, 64, 32, 1
    w = [_bits((torch.from_numpy(rng.standard_normal((d, d))) * 0.2).to(torch.bfloat16)) for _ in range(L)]
    x = _bits(torch.from_numpy(rng.standard_normal((T, d))).to(torch.bfloat16))
    tgt = _bits(torch.from_numpy(rng.standard_normal((T, d))).to(torch.bfloat16))
    jit = S.OracleStack(w, x, tgt, lr=0.1)
    his = S.OracleStack(w, x, tgt, lr=0.1, history=True, margin=margin)
    r0j, r0h = jit.step(0), his.step(0)
    assert np.array_equal(r0j["bias"], r0h["bias"]) and r0j["loss"] == r0h["loss"]
    prev = r0h["amax"]
    for step in (1, 2, 3):
        r = his.step(step)
        for l in range(L):
            assert r["bias"][l, 0] == O.scaling_bias(r["amax"][l, 0], O.E4)
            assert r["bias"][l, 1] == O.scaling_bias(prev[l, 1], O.E4) - margin
            assert r["bias"][l, 2] == O.scaling_bias(prev[l, 2], O.E5) - margin
            assert np.array_equal(r["x8"][l], O.cast(r["x"][l], int(r["bias"][l, 1]) + 1, O.N_E4))
            assert np.array_equal(r["g8"][l], O.cast(r["g"][l], int(r["bias"][l, 2]), O.N_E5))
            assert r["amax"][l, 1] == O.amax(r["x"][l]) and r["amax"][l, 2] == O.amax(r["g"][l])
        prev = r["amax"]
    # a tensor that outgrows its history clips at the format's maximum instead of overflowing
    big = S.OracleStack(w, x, tgt, lr=0.1, history=True, margin=0)
    big.step(0)
    big.prev_amax[0, 1] /= 64.0          # pretend the input was 64 times smaller at the previous step
    r = big.step(1)
    dec = np.abs(O.decode_table(O.N_E4)[r["x8"][0]])
    assert dec.max() == 448.0 and (dec == 448.0).sum() > 1


def test_swiglu_and_its_backward_against_torch_float64():
    """SwiGLU on the 32-block layout against torch's float64 silu and autograd on de-interleaved tensors."""
    rng = np.random.default_rng(11)
    T, F = 24, 96
    gate = torch.from_numpy(rng.standard_normal((T, F)) * 3).to(torch.bfloat16)
    up = torch.from_numpy(rng.standard_normal((T, F))).to(torch.bfloat16)
    gate[0, :6] = torch.tensor([-100.0, -60.0, -20.0, 0.0, 30.0, 90.0], dtype=torch.bfloat16)
    from paper_2309_17224_b200.inputs import interleave32
    y = interleave32(gate.T.contiguous(), up.T.contiguous()).T.contiguous()      # [T, 2F] in blocks of 32 columns
    assert torch.equal(y[:, :32], gate[:, :32]) and torch.equal(y[:, 32:64], up[:, :32]) and torch.equal(y[:, 64:96], gate[:, 32:64])
    g64 = gate.to(torch.float64).clone().requires_grad_(True)
    u64 = up.to(torch.float64).clone().requires_grad_(True)
    z = torch.nn.functional.silu(g64) * u64
    want = z.detach().to(torch.float32).to(torch.bfloat16)
    got = S.swiglu_bits(_bits(y))
    assert np.abs(_ord(got) - _ord(_bits(want))).max() <= 1
    dz = torch.from_numpy(rng.standard_normal((T, F)))
    z.backward(dz)
    back = S.swiglu_backward(dz.numpy(), _bits(y))
    gi, ui = S._blocks32(2 * F)
    np.testing.assert_allclose(back[:, gi], g64.grad.numpy(), rtol=1e-11, atol=1e-300)
    np.testing.assert_allclose(back[:, ui], u64.grad.numpy(), rtol=1e-11, atol=1e-300)
