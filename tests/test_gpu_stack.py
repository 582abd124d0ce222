"""Config 5, the dynamic-scaling stress run: 200 SGD steps of a 24-layer
stack of FP8 linears (d = 1024, 4096 tokens) whose input scale drifts as
2^(8 sin(step/20)).

What is compared with what:
  * every step: the bias of the first layer's input against the oracle's bias
    of the seeded, drifted input (the drift law);
  * steps 0, 1, 50, 199: the first layer's input bytes against the oracle's cast;
  * steps 0, 1, 50 and 199, layers 0, 12 and 23, teacher-forced: the run keeps
    the bf16 tensors each linear actually saw at that step (input, weight after
    that many SGD updates, output gradient) and everything the library made of
    them; the oracle is given those same bf16 tensors and must agree on amax,
    bias and FP8 bytes bit for bit and on Y, dX, dW to one bf16 ulp.  (A matmul
    output that differs within tolerance can move the next tensor's amax across
    a power of two, so two free-running trajectories cannot be compared byte for
    byte; each op on identical inputs can.)
  * steps 0 and 1: the oracle also runs the whole trajectory from the seeded
    tensors.  Each GPU linear is given the ORACLE's tensors for three layers of
    the stack and must reproduce the oracle's bytes and outputs; the
    free-running GPU trajectory must agree with the oracle's in loss and (away
    from power-of-two boundaries) in every bias;
  * steps 50 and 199 besides: the defining inequality of Eq. 3 for every bias
    the GPU produced, finite loss, no device time-out.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle as O
from oracle import stack as OS
from helpers import assert_bf16_within_one_ulp, assert_codes_equal, bf16_from_bits, bits_of, u8
from paper_2309_17224_b200 import inputs as I

pytestmark = pytest.mark.gpu

CHECK_STEPS = (0, 1, 50, 199)
LAYERS, D, TOKENS, STEPS = 24, 1024, 4096, 200
SNAP_LAYERS = (0, LAYERS // 2, LAYERS - 1)


@pytest.fixture(scope="module")
def run():
    from paper_2309_17224_b200 import fp8lin, stack
    ctx = fp8lin.Context(0)
    st = stack.Fp8Stack(ctx, layers=LAYERS, d=D, tokens=TOKENS, log_steps=STEPS)
    seeded = {"w": [bits_of(w.to(torch.bfloat16)) for w in st.w32], "x_base": bits_of(st.x_base),
              "target": bits_of(st.target)}
    trace = []
    x8_at, snaps = {}, {}
    for step in range(STEPS):
        r = st.step(step, snap_layers=SNAP_LAYERS if step in CHECK_STEPS else ())
        trace.append(r)
        if step in CHECK_STEPS:
            x8_at[step] = u8(st.x8[0])
            snaps[step] = {l: {k: v.cpu() for k, v in d.items()} for l, d in st.snap.items()}
    torch.cuda.synchronize()
    flags = ctx.device_flags(clear=True)
    out = {"lib": fp8lin, "ctx": ctx, "stack": st, "seeded": seeded, "x8_at": x8_at, "flags": flags, "snaps": snaps,
           "loss": [float(r["loss"].item()) for r in trace],
           "bias": np.stack([r["bias"].cpu().numpy() for r in trace]),
           "amax": np.stack([r["amax"].cpu().numpy() for r in trace])}
    yield out
    ctx.close()


def test_fused_activation_variant_tracks_the_plain_run(run):
    """GELU in the matmul epilogue + amax from the epilogue (one quantisation pass per activation): the first
    step's loss and biases must agree with the unfused run's (same arithmetic, different kernels)."""
    from paper_2309_17224_b200 import stack
    st = stack.Fp8Stack(run["ctx"], layers=LAYERS, d=D, tokens=TOKENS, fused_activation=True)
    for step in (0, 1):
        r = st.step(step)
        assert abs(float(r["loss"].item()) - run["loss"][step]) <= 1e-3 * run["loss"][step]
        same = (r["bias"].cpu().numpy() == run["bias"][step])
        assert same.mean() >= 0.97
    assert run["ctx"].device_flags(clear=True) & run["lib"].FLAG_TIMEOUT == 0


def test_bias_log_and_bias_modes(run, tmp_path):
    """The device-side log holds one record per tensor and step, equal to what each step returned; the per-tensor
    mode of the bias over a window of steps (Appendix G's statistic) equals the oracle's rule on that trace; the CSV
    the harness writes carries the same numbers."""
    st = run["stack"]
    recs = st.bias_records()
    assert len(recs) == STEPS * LAYERS * 3
    names = ("W", "X", "dY")
    for step in (0, 1, 57, 199):
        for l in (0, 11, 23):
            for j in range(3):
                r = recs[(step * LAYERS + l) * 3 + j]
                assert r == (step, l, names[j], float(run["amax"][step, l, j]), int(run["bias"][step, l, j]))
    for lo, hi in ((0, STEPS - 1), (40, 79), (199, 199)):
        modes = st.bias_modes(lo, hi).cpu().numpy()
        for l in range(LAYERS):
            for j in range(3):
                assert tuple(modes[l, j]) == O.bias_mode(run["bias"][lo:hi + 1, l, j]), (lo, hi, l, j)
    # weights keep one bias almost always, the input's bias follows the drift (Appendix I: weights and activations
    # nearly static, here the input is driven on purpose)
    whole = st.bias_modes(0, STEPS - 1).cpu().numpy()
    assert whole[:, 0, 1].min() >= 0.9 * STEPS and whole[0, 1, 1] < 0.5 * STEPS
    path = tmp_path / "bias.csv"
    assert st.write_bias_csv(str(path)) == STEPS * LAYERS * 3
    lines = path.read_text().splitlines()
    assert lines[0] == "step,layer,tensor,amax,bias" and len(lines) == 1 + STEPS * LAYERS * 3
    step, layer, tensor, amax, bias = lines[1 + (57 * LAYERS + 11) * 3 + 2].split(",")
    assert (int(step), int(layer), tensor, float(amax), int(bias)) == (57, 11, "dY", float(run["amax"][57, 11, 2]),
                                                                       int(run["bias"][57, 11, 2]))


def test_no_timeouts_and_finite_losses(run):
    assert run["flags"] & run["lib"].FLAG_TIMEOUT == 0
    assert np.all(np.isfinite(run["loss"]))


def test_first_layer_input_bias_follows_the_drift_law(run):
    """b_x of layer 0 at every step equals the oracle's bias for the seeded input scaled by 2^(8 sin(step/20))."""
    moves = set()
    for step in range(STEPS):
        xb = OS.step_input_bits(run["seeded"]["x_base"], step)
        a = O.amax(xb)
        b = O.scaling_bias(a, O.E4)
        assert run["amax"][step, 0, 1] == a and run["bias"][step, 0, 1] == b, step
        moves.add(b)
        if step in CHECK_STEPS:
            assert_codes_equal(run["x8_at"][step], O.cast(xb, b + 1, O.N_E4), O.N_E4)
    assert max(moves) - min(moves) >= 14   # the drift spans 2^-8 .. 2^8


def test_every_bias_satisfies_the_inequality_of_eq3(run):
    """amax * 2^b <= max_num < amax * 2^(b+1), exact arithmetic, for every tensor at the checked steps."""
    for step in CHECK_STEPS:
        for l in range(LAYERS):
            for j, mx in ((0, 240), (1, 240), (2, 57344)):
                a = Fraction(float(run["amax"][step, l, j]))
                b = int(run["bias"][step, l, j])
                assert a > 0
                assert a * Fraction(2) ** b <= mx < a * Fraction(2) ** (b + 1), (step, l, j)


def test_gradient_biases_move_with_the_drift(run):
    """The gradient format needs its own, far larger biases, and they move."""
    bg = run["bias"][:, :, 2]
    assert bg.min() > run["bias"][:, :, 0].max()
    assert len(np.unique(bg[:, 0])) >= 3


@pytest.mark.parametrize("step", CHECK_STEPS)
def test_checked_steps_teacher_forced_against_the_oracle(run, step):
    """Config 5's comparison at steps 0, 1, 50 and 199: for the first, the middle and the last layer, the oracle
    quantises the very bf16 tensors the GPU linear saw at that step and multiplies the resulting bytes; amax, bias
    and bytes must be equal, Y, dX and dW within one bf16 ulp."""
    for l in SNAP_LAYERS:
        sn = run["snaps"][step][l]
        got_amax, got_bias = sn["amax"].tolist(), sn["bias"].tolist()
        aw, bw, w8 = O.quantise(bits_of(sn["w"]), O.E4)
        ax, bx, x8 = O.quantise(bits_of(sn["x"]), O.E4)
        ag, bg, g8 = O.quantise(bits_of(sn["g"]), O.E5)
        assert got_amax == [aw, ax, ag] and got_bias == [bw, bx, bg], (step, l)
        assert_codes_equal(u8(sn["w8"]), w8, O.N_E4)
        assert_codes_equal(u8(sn["x8"]), x8, O.N_E4)
        assert_codes_equal(u8(sn["g8"]), g8, O.N_E5)
        assert_bf16_within_one_ulp(bits_of(sn["y"]), O.linear_fwd_np(x8, bx + 1, w8, bw + 1))
        assert_bf16_within_one_ulp(bits_of(sn["dx"]), O.linear_dgrad_np(g8, bg, w8, bw + 1))
        assert_bf16_within_one_ulp(bits_of(sn["dw"]), O.linear_wgrad_np(g8, bg, x8, bx + 1))
    if step >= 50:
        assert run["bias"][step, 0, 1] != run["bias"][0, 0, 1]   # the input scale has drifted since step 0


def test_steps_0_and_1_against_the_oracle_trajectory(run):
    lib, ctx = run["lib"], run["ctx"]
    sd = run["seeded"]
    orc = OS.OracleStack(sd["w"], sd["x_base"], sd["target"], lr=1e-3)
    dev = dict(device="cuda")
    for step in (0, 1):
        rec = orc.step(step)
        # free-running GPU trajectory against the oracle's
        assert abs(run["loss"][step] - rec["loss"]) <= 2e-3 * rec["loss"]
        same = run["bias"][step] == rec["bias"]
        assert same.mean() >= 0.95
        for l, j in np.argwhere(~same):
            # a bias may differ only where the amax sits at a power-of-two boundary of max_num
            mx = 57344.0 if j == 2 else 240.0
            frac = np.log2(mx / rec["amax"][l, j]) % 1.0
            assert min(frac, 1.0 - frac) < 0.02, (step, l, j)
        # each GPU linear fed the oracle's tensors
        amax = torch.zeros(3, dtype=torch.float32, **dev)
        bias = torch.zeros(3, dtype=torch.int32, **dev)
        u8k = dict(dtype=torch.uint8, **dev)
        for l in (0, LAYERS // 2, LAYERS - 1):
            x = bf16_from_bits(rec["x"][l], "cuda")
            w = bf16_from_bits(rec["w"][l], "cuda")
            g = bf16_from_bits(rec["g"][l], "cuda")
            x8, x8t = torch.empty((TOKENS, D), **u8k), torch.empty((D, TOKENS), **u8k)
            w8, w8t = torch.empty((D, D), **u8k), torch.empty((D, D), **u8k)
            g8, g8t = torch.empty((TOKENS, D), **u8k), torch.empty((D, TOKENS), **u8k)
            ctx.cast_e4(w, None, d_amax_out=amax[0:1], d_bias_out=bias[0:1], y=w8, y_t=w8t)
            ctx.cast_e4(x, None, d_amax_out=amax[1:2], d_bias_out=bias[1:2], y=x8, y_t=x8t)
            ctx.cast_e5(g, None, d_amax_out=amax[2:3], d_bias_out=bias[2:3], y=g8, y_t=g8t)
            assert bias.tolist() == rec["bias"][l].tolist() and amax.tolist() == rec["amax"][l].tolist()
            assert_codes_equal(u8(w8), rec["w8"][l], O.N_E4)
            assert_codes_equal(u8(x8), rec["x8"][l], O.N_E4)
            assert_codes_equal(u8(g8), rec["g8"][l], O.N_E5)
            assert np.array_equal(u8(x8t), rec["x8"][l].T) and np.array_equal(u8(g8t), rec["g8"][l].T)
            y = torch.empty((TOKENS, D), dtype=torch.bfloat16, **dev)
            dx = torch.empty((TOKENS, D), dtype=torch.bfloat16, **dev)
            dw = torch.empty((D, D), dtype=torch.bfloat16, **dev)
            ctx.linear_fwd(x8, bias[1:2], w8, bias[0:1], y)
            ctx.linear_dgrad(g8, bias[2:3], None, w8t, bias[0:1], dx)
            ctx.linear_wgrad(None, g8t, bias[2:3], None, x8t, bias[1:2], dw, TOKENS)
            assert_bf16_within_one_ulp(bits_of(y), rec["y"][l])
            assert_bf16_within_one_ulp(bits_of(dx), rec["dx"][l])
            assert_bf16_within_one_ulp(bits_of(dw), rec["dw"][l])
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_history_scaling_stack_against_the_oracle_trajectory():
    """Amax-history scaling (Section 3): activations and gradients are quantised by the producing matmul's
    epilogue with the previous step's bias minus a margin of one.  A smaller stack, so that the oracle can
    follow it for six steps; same agreement bars as the just-in-time run, and nothing may clip: the input
    grows by at most 2^0.4 per step, inside the margin."""
    from paper_2309_17224_b200 import fp8lin, stack
    L, d, T, steps, margin = 6, 512, 1024, 6, 1
    ctx = fp8lin.Context(0)
    try:
        st = stack.Fp8StackHistory(ctx, margin=margin, layers=L, d=d, tokens=T)
        orc = OS.OracleStack([bits_of(w.to(torch.bfloat16)) for w in st.w32], bits_of(st.x_base), bits_of(st.target),
                             lr=1e-3, history=True, margin=margin)
        for step in range(steps):
            r = st.step(step, snap_layers=(0, L // 2, L - 1) if step == steps - 1 else ())
            flags = ctx.device_flags(clear=True)
            assert flags & fp8lin.FLAG_TIMEOUT == 0
            if step > 0:
                assert flags & fp8lin.FLAG_SATURATED == 0
            if step == steps - 1:
                # teacher-forced: the oracle multiplies the bytes the GPU matmuls were given at this step, under the
                # biases they were given, and quantises the weight the GPU quantised
                for l, sn in st.snap.items():
                    sn = {k: v.cpu() for k, v in sn.items()}
                    aw, bw, w8 = O.quantise(bits_of(sn["w"]), O.E4)
                    assert int(sn["bias_w"].item()) == bw
                    assert_codes_equal(u8(sn["w8"]), w8, O.N_E4)
                    bx, bg = int(sn["bias_x"].item()), int(sn["bias_g"].item())
                    assert_bf16_within_one_ulp(bits_of(sn["y"]), O.linear_fwd_np(u8(sn["x8"]), bx + 1, w8, bw + 1))
                    assert_bf16_within_one_ulp(bits_of(sn["dw"]), O.linear_wgrad_np(u8(sn["g8"]), bg, u8(sn["x8"]), bx + 1))
            rec = orc.step(step)
            assert abs(float(r["loss"].item()) - rec["loss"]) <= 2e-3 * rec["loss"], step
            got = r["bias"].cpu().numpy()
            same = got == rec["bias"]
            assert same.mean() >= 0.9, (step, same.mean())
            for l, j in np.argwhere(~same):
                mx = 57344.0 if j == 2 else 240.0
                src = orc_prev_amax[l, j] if (step > 0 and j > 0) else rec["amax"][l, j]
                frac = np.log2(mx / src) % 1.0
                assert min(frac, 1.0 - frac) < 0.02, (step, l, j)
            if step > 0:
                # the biases in use are the previous step's, one below what Eq. 3 gives for that amax
                for l in range(L):
                    for j, kind in ((1, O.E4), (2, O.E5)):
                        assert rec["bias"][l, j] == O.scaling_bias(float(orc_prev_amax[l, j]), kind) - margin
            orc_prev_amax = rec["amax"].copy()
    finally:
        ctx.close()
