"""GPU parity: fp8_cast_group (FP8-AMAX of several tensors in two launches) against the CPU oracle, bit for bit,
in both modes (just in time; one pass with verified bias guesses), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_codes_equal, bits_of, u8
from paper_2309_17224_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2309_17224_b200 import fp8lin
    return fp8lin


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0)
    yield c
    c.close()


def _np_input(x):
    """What the oracle reads: bf16 as bit patterns, fp16 / fp32 as numpy arrays."""
    return bits_of(x) if x.dtype == torch.bfloat16 else x.cpu().numpy()


class Tensors:
    """A group: inputs, per-tensor outputs, the item list, the oracle's answers."""

    def __init__(self, specs, seed=1):
        self.x, self.kind, self.margin = [], [], []
        for i, (rows, cols, std, kind, dtype, margin) in enumerate(specs):
            t = I.normal_bf16(rows, cols, std, seed, 100 + i, "cuda", outlier_frac=0.01, outlier_scale=30.0)
            self.x.append(t if dtype == torch.bfloat16 else t.to(dtype))
            self.kind.append(kind)
            self.margin.append(margin)
        n = len(specs)
        self.amax = torch.full((n,), -1.0, dtype=torch.float32, device="cuda")
        self.bias = torch.zeros(n, dtype=torch.int32, device="cuda")
        self.y = [torch.full(x.shape, 0xAA, dtype=torch.uint8, device="cuda") for x in self.x]
        self.ref = [O.quantise(_np_input(x), k, O.CONV_PAPER, m) for x, k, m in zip(self.x, self.kind, self.margin)]

    def items(self):
        return [(k, x, self.amax[i:i + 1], self.bias[i:i + 1], self.y[i], m)
                for i, (k, x, m) in enumerate(zip(self.kind, self.x, self.margin))]

    def check(self):
        assert self.amax.tolist() == [r[0] for r in self.ref]
        assert self.bias.tolist() == [r[1] for r in self.ref]
        for y, r, k in zip(self.y, self.ref, self.kind):
            assert_codes_equal(u8(y), r[2], O.native_format(k))

    def scribble(self):
        self.amax.fill_(-1.0)
        for y in self.y:
            y.fill_(0xAA)


BF = torch.bfloat16
SPECS = [
    (256, 768, 1.0, O.E4, BF, 0),          # config-1 sizes
    (768, 768, 0.02, O.E4, BF, 0),
    (256, 768, 1e-3, O.E5, BF, 3),
    (1, 5, 2.0, O.E4, BF, 0),              # less than one output vector: tail only
    (3, 1001, 1e-5, O.E5, BF, 0),          # ragged tail behind whole vectors
    (1024, 4096, 1.0, O.E4, BF, 0),        # many chunks
    (130, 8192 * 3 + 16, 0.5, O.E5, BF, 1),
    (64, 64, 2.0 ** -120, O.E4, BF, 0),    # shift beyond one float factor
    (64, 64, 2.0 ** 100, O.E5, BF, 0),
]


def test_group_just_in_time_equals_the_oracle_per_tensor(ctx, lib):
    g = Tensors(SPECS)
    ctx.device_flags(clear=True)
    before = lib.launch_count()
    ctx.cast_group(g.items())
    assert lib.launch_count() - before == 2            # one amax pass, one cast pass for the whole group
    g.check()
    # a second call on the same slots (every reduction slot must have been left clean)
    g.scribble()
    ctx.cast_group(lib.group_items(g.items()))
    g.check()
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_group_predicted_is_exact_whatever_the_guesses(ctx, lib):
    g = Tensors(SPECS, seed=2)
    truth = torch.tensor([r[1] for r in g.ref], dtype=torch.int32, device="cuda")
    n = len(SPECS)
    ctx.prediction_stats(clear=True)
    for label, guesses in (("all right", truth.clone()),
                           ("all wrong", truth + 1),
                           ("mixed", truth + torch.tensor([0, 1, 0, -2, 0, 0, 5, 0, -1], dtype=torch.int32, device="cuda")),
                           ("absurd", torch.tensor([2 ** 31 - 1, -2 ** 31, 400, -400, 0, 127, -127, 1000, -1000],
                                                   dtype=torch.int32, device="cuda"))):
        g.scribble()
        g.bias.copy_(guesses)
        ctx.cast_group(g.items(), predicted=True)
        g.check()
        hits, misses = ctx.prediction_stats(clear=True)
        assert hits == int((guesses == truth).sum().item()) and hits + misses == n, label
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_group_saturation_flag_follows_the_true_bias_only(ctx, lib):
    """Clipping under a wrong guess must not raise FP8_FLAG_SATURATED; clipping under the true bias must (a tensor
    whose scaled amax rounds to the paper format's 240 code)."""
    x = (torch.randn((64, 512), device="cuda") * 10.0).clamp(-100, 100).to(BF)
    amax, bias = torch.zeros(1, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
    for top, guess, expect in ((100.0, 5, False), (100.0, 1, False), (236.0, 0, True), (236.0, 3, True)):
        x[7, 7] = top
        ctx.device_flags(clear=True)
        bias.fill_(guess)
        ctx.cast_group([(lib.E4, x, amax, bias, y)], predicted=True)
        a, b, ref = O.quantise(bits_of(x), O.E4)
        assert (float(amax.item()), int(bias.item())) == (a, b)
        assert_codes_equal(u8(y), ref, O.N_E4)
        assert bool(ctx.device_flags(clear=True) & lib.FLAG_SATURATED) == expect, (top, guess)


def test_group_mixed_types_strided_members_and_more_than_one_round(ctx, lib):
    specs = [(96, 520, 1.0, O.E4, torch.float16, 0), (96, 520, 1.0, O.E4, torch.float32, 0), (33, 77, 0.1, O.E5, BF, 0)]
    specs += [(40 + i, 256, 0.3 * (i + 1), O.E4 if i % 2 else O.E5, BF, i % 3) for i in range(20)]   # > 16 of one type
    g = Tensors(specs, seed=3)
    # one member handed over as a strided view: it must take the single-tensor path and still come out right
    wide = I.normal_bf16(50, 300, 1.0, 9, 9, "cuda")
    view = wide[:, 8:264]
    va, vb = torch.zeros(1, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
    vy = torch.empty((50, 256), dtype=torch.uint8, device="cuda")
    items = g.items()
    items.insert(5, (lib.E4, view, va, vb, vy))
    for predicted in (False, True):
        g.scribble()
        vy.fill_(0)
        ctx.cast_group(items, predicted=predicted)
        g.check()
        a, b, ref = O.quantise(bits_of(view), O.E4)
        assert (float(va.item()), int(vb.item())) == (a, b)
        assert_codes_equal(u8(vy), ref, O.N_E4)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_group_special_values(ctx, lib):
    x0 = torch.zeros((16, 64), dtype=BF, device="cuda")                     # amax 0 -> bias 0, flag
    x1 = torch.randn((16, 64), device="cuda").to(BF); x1[3, 3] = float("inf")
    x2 = torch.randn((16, 64), device="cuda").to(BF); x2[0, 1] = float("nan")
    xs = [x0, x1, x2]
    amax = torch.zeros(3, device="cuda")
    bias = torch.full((3,), 7, dtype=torch.int32, device="cuda")
    ys = [torch.empty(x.shape, dtype=torch.uint8, device="cuda") for x in xs]
    for predicted in (False, True):
        ctx.device_flags(clear=True)
        ctx.cast_group([(lib.E4, x, amax[i:i + 1], bias[i:i + 1], ys[i]) for i, x in enumerate(xs)], predicted=predicted)
        flags = ctx.device_flags(clear=True)
        assert flags & lib.FLAG_ZERO_AMAX and flags & lib.FLAG_NONFINITE_AMAX
        for i, x in enumerate(xs):
            a, b, ref = O.quantise(bits_of(x), O.E4)
            got = float(amax[i].item())
            assert (np.isnan(a) and np.isnan(got)) or a == got
            assert int(bias[i].item()) == b == 0
            assert_codes_equal(u8(ys[i]), ref, O.N_E4)


def test_group_single_passes(ctx, lib):
    """FP8_GROUP_AMAX_ONLY writes amax and bias and leaves the bytes alone; FP8_GROUP_CAST_ONLY casts with the
    biases it is given (a constant bias per tensor: FP8-CSCALE) and leaves amax alone."""
    g = Tensors(SPECS, seed=4)
    ctx.cast_group(g.items(), mode=lib.GROUP_AMAX_ONLY)
    assert g.amax.tolist() == [r[0] for r in g.ref] and g.bias.tolist() == [r[1] for r in g.ref]
    assert all(bool((y == 0xAA).all()) for y in g.y)
    no_y = [(k, x, a, b, None, m) for (k, x, a, b, y, m) in g.items()]
    g.amax.fill_(-1.0)
    ctx.cast_group(no_y, mode=lib.GROUP_AMAX_ONLY)
    assert g.amax.tolist() == [r[0] for r in g.ref]
    given = torch.tensor([3, -2, 20, 0, 17, 1, 9, 115, -95], dtype=torch.int32, device="cuda")
    g.bias.copy_(given)
    g.amax.fill_(-5.0)
    ctx.cast_group(g.items(), mode=lib.GROUP_CAST_ONLY)
    assert bool((g.amax == -5.0).all()) and torch.equal(g.bias, given)
    for x, y, k, b in zip(g.x, g.y, g.kind, given.tolist()):
        want = O.cast(_np_input(x), b + O.delta(k, O.CONV_PAPER), O.native_format(k))
        assert_codes_equal(u8(y), want, O.native_format(k))
    ctx.device_flags(clear=True)


def test_group_argument_errors(ctx, lib):
    x = torch.zeros((8, 16), dtype=BF, device="cuda")
    a, b = torch.zeros(1, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.zeros((8, 16), dtype=torch.uint8, device="cuda")
    arr = lib.group_items([(lib.E4, x, a, b, y)])
    raw = lib.raw()
    assert raw.fp8_cast_group(ctx._h, arr, 0, 0, 0, None) == lib.ERR_SHAPE
    assert raw.fp8_cast_group(ctx._h, None, 1, 0, 0, None) == lib.ERR_NULL
    assert raw.fp8_cast_group(ctx._h, arr, 1, 5, 0, None) == lib.ERR_DTYPE
    assert raw.fp8_cast_group(ctx._h, arr, 1, 0, 4, None) == lib.ERR_DTYPE
    arr[0].fmt = 9
    assert raw.fp8_cast_group(ctx._h, arr, 1, 0, 0, None) == lib.ERR_DTYPE
    arr[0].fmt = 0
    arr[0].y = None
    assert raw.fp8_cast_group(ctx._h, arr, 1, 0, 0, None) == lib.ERR_NULL


def test_group_at_benchmark_size_matches_the_single_tensor_calls(ctx, lib):
    """The twelve tensors of one Llama-2-7B step in one group, both modes: identical bytes, amax and biases to
    fp8_cast_e4 / _e5 per tensor (which the other tests hold against the oracle at this size)."""
    wl = I.WORKLOADS["c3_llama7b"]
    xs, kinds = [], []
    for li in range(len(wl.layers)):
        t = I.layer_tensors(wl, li, device="cuda")
        xs += [t["w"], t["x"], t["g"]]
        kinds += [lib.E4, lib.E4, lib.E5]
    n = len(xs)
    amax, bias = torch.zeros(n, device="cuda"), torch.zeros(n, dtype=torch.int32, device="cuda")
    amax1, bias1 = torch.zeros(n, device="cuda"), torch.zeros(n, dtype=torch.int32, device="cuda")
    ys = [torch.empty(x.shape, dtype=torch.uint8, device="cuda") for x in xs]
    items = lib.group_items([(k, x, amax[i:i + 1], bias[i:i + 1], ys[i]) for i, (k, x) in enumerate(zip(kinds, xs))])
    ctx.cast_group(items)
    got = [y.clone() for y in ys]
    y1 = torch.empty(max(x.numel() for x in xs), dtype=torch.uint8, device="cuda")
    for i, (k, x) in enumerate(zip(kinds, xs)):
        yy = y1[:x.numel()].view(x.shape)
        (ctx.cast_e4 if k == lib.E4 else ctx.cast_e5)(x, None, d_amax_out=amax1[i:i + 1], d_bias_out=bias1[i:i + 1], y=yy)
        assert torch.equal(got[i], yy)
    assert torch.equal(amax, amax1) and torch.equal(bias, bias1)
    ctx.prediction_stats(clear=True)
    for y in ys:
        y.zero_()
    ctx.cast_group(items, predicted=True)          # the biases of the first call are the guesses: all hold
    assert ctx.prediction_stats(clear=True) == (n, 0)
    for i in range(n):
        assert torch.equal(got[i], ys[i])
    assert torch.equal(amax, amax1) and torch.equal(bias, bias1)
