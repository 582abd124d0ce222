"""GPU parity of fp8_linear_group (several independent matmuls in one launch) against the CPU oracle and against
the three single-matmul calls it stands for.

Every member's output must meet the bars of its own entry point (FP32: 2^-14 * sum_k |a*b|; bf16: one ulp of the
oracle's rounding).  Against the single calls the outputs may differ by the order of the FP32 accumulation only
(another tile shape walks the contraction in another direction): at most one bf16 step at the tensor's largest
magnitude.
"""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import assert_bf16_within_one_ulp, assert_gemm_close, bits_of, tile_sample_positions
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


class Layer:
    """One linear's three tensors quantised on the GPU (row-major bytes) and by the oracle."""

    def __init__(self, ctx, T, K, N, seed, conv=O.CONV_PAPER, tensors=None):
        self.T, self.K, self.N = T, K, N
        if tensors is None:
            x = I.normal_bf16(T, K, 1.0, seed, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0)
            w = I.normal_bf16(N, K, 0.02, seed, 2, "cuda")
            g = I.normal_bf16(T, N, 1e-3, seed, 3, "cuda")
        else:
            x, w, g = tensors
        self.bias = torch.zeros(3, dtype=torch.int32, device="cuda")
        amax = torch.zeros(3, dtype=torch.float32, device="cuda")
        self.x8, self.w8, self.g8 = (torch.empty(t.shape, dtype=torch.uint8, device="cuda") for t in (x, w, g))
        ctx.cast_e4(w, None, conv=conv, d_amax_out=amax[0:1], d_bias_out=self.bias[0:1], y=self.w8)
        ctx.cast_e4(x, None, conv=conv, d_amax_out=amax[1:2], d_bias_out=self.bias[1:2], y=self.x8)
        ctx.cast_e5(g, None, conv=conv, d_amax_out=amax[2:3], d_bias_out=self.bias[2:3], y=self.g8)
        _, bw, self.rw = O.quantise(bits_of(w), O.E4, conv)
        _, bx, self.rx = O.quantise(bits_of(x), O.E4, conv)
        _, bg, self.rg = O.quantise(bits_of(g), O.E5, conv)
        assert self.bias.tolist() == [bw, bx, bg]
        for got, want in ((self.w8, self.rw), (self.x8, self.rx), (self.g8, self.rg)):
            assert np.array_equal(got.cpu().numpy(), want)
        self.sw, self.sx, self.sg = bw + O.delta(O.E4, conv), bx + O.delta(O.E4, conv), bg + O.delta(O.E5, conv)

    def outputs(self, dt):
        return [torch.full(s, float("nan"), dtype=dt, device="cuda")
                for s in ((self.T, self.N), (self.T, self.K), (self.N, self.K))]

    def items(self, lib, outs, bias_vec=None, amax=None):
        b = self.bias
        return [(lib.MATMUL_FWD, self.x8, b[1:2], self.w8, b[0:1], outs[0], bias_vec, amax[0:1] if amax is not None else None),
                (lib.MATMUL_DGRAD, self.g8, b[2:3], self.w8, b[0:1], outs[1], None, amax[1:2] if amax is not None else None),
                (lib.MATMUL_WGRAD, self.g8, b[2:3], self.x8, b[1:2], outs[2])]

    def single_calls(self, ctx, outs, bias_vec=None, conv=O.CONV_PAPER):
        b = self.bias
        ctx.linear_fwd(self.x8, b[1:2], self.w8, b[0:1], outs[0], bias_vec=bias_vec, conv=conv)
        ctx.linear_dgrad(self.g8, b[2:3], self.w8, None, b[0:1], outs[1], conv=conv)
        ctx.linear_wgrad(self.g8, None, b[2:3], self.x8, None, b[1:2], outs[2], self.T, conv=conv)

    def oracle(self, bias_vec=None):
        return (O.linear_fwd(self.rx, self.sx, self.rw, self.sw, bias_vec=bias_vec),
                O.linear_dgrad(self.rg, self.sg, self.rw, self.sw), O.linear_wgrad(self.rg, self.sg, self.rx, self.sx))


def _close_to_single_call(got, one):
    """Both meet the oracle's bar on their own; against each other they may differ by the order of the FP32 sums:
    no more than one bf16 step at the largest magnitude of the tensor."""
    a, b = got.float(), one.float()
    return float((a - b).abs().max()) <= float(b.abs().max()) * 2.0 ** -7


GROUPS = [
    [(400, 1040, 784)],                                            # one layer: three matmuls of three shapes
    [(256, 768, 768), (272, 8208, 304), (144, 272, 528)],          # ragged in every dimension, one long contraction
    [(384, 2048, 1024), (640, 2048, 512), (512, 4096, 1536)],      # every member fits the 512-column tile
    [(1024, 512, 2560), (300, 272, 4112), (2048, 1024, 256), (130, 144, 272), (200, 4096, 144), (272, 528, 144)],   # 18 matmuls: more than one launch holds
]


@pytest.mark.parametrize("shapes", GROUPS)
@pytest.mark.parametrize("conv", [O.CONV_PAPER, O.CONV_NATIVE])
def test_group_matches_oracle_and_single_calls(ctx, lib, shapes, conv):
    layers = [Layer(ctx, T, K, N, 100 + i, conv) for i, (T, K, N) in enumerate(shapes)]
    bvs = [(torch.randn(L.N, device="cuda") * 0.1).to(torch.bfloat16) for L in layers]
    refs = [L.oracle(bias_vec=bv.double().cpu().numpy()) for L, bv in zip(layers, bvs)]
    for dt in (torch.float32, torch.bfloat16):
        outs = [L.outputs(dt) for L in layers]
        single = [L.outputs(dt) for L in layers]
        amax = torch.full((len(layers), 2), -1.0, dtype=torch.float32, device="cuda")
        items = [it for i, (L, o, bv) in enumerate(zip(layers, outs, bvs)) for it in L.items(lib, o, bv, amax[i])]
        n0 = lib.launch_count()
        ctx.linear_group(items, conv=conv)
        launched = lib.launch_count() - n0
        assert launched == 1 if len(items) <= 16 else launched >= len(items), launched
        for L, o, bv in zip(layers, single, bvs):
            L.single_calls(ctx, o, bias_vec=bv, conv=conv)
        torch.cuda.synchronize()
        for i, (L, o, s, ref) in enumerate(zip(layers, outs, single, refs)):
            for got, one, want in zip(o, s, ref):
                if dt == torch.float32:
                    assert_gemm_close(got.cpu().numpy(), want)
                else:
                    assert_bf16_within_one_ulp(bits_of(got), want)
                    assert _close_to_single_call(got, one)
            assert float(amax[i, 0].item()) == float(o[0].float().abs().max().item())
            assert float(amax[i, 1].item()) == float(o[1].float().abs().max().item())
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_ragged_last_columns_survive_a_busy_gpu(ctx, lib):
    """A tile that hangs over the last column stores only its first chunks; the staging slabs of the chunks it skips
    must not be rewritten while the last real store still reads them.  On an idle GPU the store wins the race by a
    wide margin; with 160 tiles of nine problems in flight it did not (zeros in the last 16 columns of a weight
    gradient in one launch out of twenty).  Two hundred launches, every one bit-identical to the first and that one
    within the oracle's bars."""
    layers = [Layer(ctx, T, K, N, 500 + i) for i, (T, K, N) in enumerate([(256, 768, 768), (272, 8208, 304), (144, 272, 528)])]
    refs = [L.oracle() for L in layers]
    first = None
    for rnd in range(200):
        outs = [L.outputs(torch.float32) for L in layers]
        ctx.linear_group([it for L, o in zip(layers, outs) for it in L.items(lib, o)])
        torch.cuda.synchronize()
        if first is None:
            first = outs
            for o, ref in zip(outs, refs):
                for got, want in zip(o, ref):
                    assert_gemm_close(got.cpu().numpy(), want)
        else:
            for a, b in zip(first, outs):
                for u, v in zip(a, b):
                    assert torch.equal(u.view(torch.int32), v.view(torch.int32)), f"launch {rnd}"
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


@pytest.mark.parametrize("dt", [torch.float32, torch.bfloat16])
def test_group_members_whose_rows_are_not_16_byte_multiples(ctx, lib, dt):
    """Outputs with N = 300 or 1030 columns cannot leave through TMA stores (rows are not multiples of 16 bytes): such
    members store from registers, inside the same launch as members that do use TMA stores."""
    members = []
    for i, (T, K, N) in enumerate([(256, 272, 300), (400, 1040, 1030), (384, 512, 768)]):
        x = I.normal_bf16(T, K, 1.0, 600 + i, 1, "cuda")
        w = I.normal_bf16(N, K, 0.02, 600 + i, 2, "cuda")
        bias = torch.zeros(2, dtype=torch.int32, device="cuda")
        amax = torch.zeros(2, dtype=torch.float32, device="cuda")
        x8, w8 = torch.empty((T, K), dtype=torch.uint8, device="cuda"), torch.empty((N, K), dtype=torch.uint8, device="cuda")
        ctx.cast_e4(x, None, d_amax_out=amax[0:1], d_bias_out=bias[0:1], y=x8)
        ctx.cast_e4(w, None, d_amax_out=amax[1:2], d_bias_out=bias[1:2], y=w8)
        _, bx, rx = O.quantise(bits_of(x), O.E4)
        _, bw, rw = O.quantise(bits_of(w), O.E4)
        y = torch.full((T, N), float("nan"), dtype=dt, device="cuda")
        members.append((x8, w8, bias, y, O.linear_fwd(rx, bx + 1, rw, bw + 1)))
    n0 = lib.launch_count()
    ctx.linear_group([(lib.MATMUL_FWD, x8, b[0:1], w8, b[1:2], y) for x8, w8, b, y, _ in members])
    assert lib.launch_count() - n0 == 1
    torch.cuda.synchronize()
    for _, _, _, y, ref in members:
        if dt == torch.float32:
            assert_gemm_close(y.cpu().numpy(), ref)
        else:
            assert_bf16_within_one_ulp(bits_of(y), ref)
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def test_group_with_a_decode_size_member_runs_the_members_own_calls(ctx, lib):
    big, small = Layer(ctx, 512, 1024, 768, 200), Layer(ctx, 16, 2048, 1280, 201)
    ob, os_ = big.outputs(torch.bfloat16), small.outputs(torch.bfloat16)
    sb, ss = big.outputs(torch.bfloat16), small.outputs(torch.bfloat16)
    # the small layer's forward and input gradient have 16 rows; its weight gradient (1280 rows) does not
    items = big.items(lib, ob) + small.items(lib, os_)
    ctx.linear_group(items)
    big.single_calls(ctx, sb)
    small.single_calls(ctx, ss)
    torch.cuda.synchronize()
    for got, one in zip(ob + os_, sb + ss):
        assert torch.equal(got.view(torch.int16), one.view(torch.int16))   # the very same launches
    for got, want in zip(os_, small.oracle()):
        assert_bf16_within_one_ulp(bits_of(got), want)


def test_group_repeated_calls_and_graph_replay(ctx, lib):
    """The item array is read during the call only; the call neither synchronises nor allocates, so it can be captured."""
    layers = [Layer(ctx, 384, 2048, 1024, 300), Layer(ctx, 640, 1024, 512, 301)]
    outs = [L.outputs(torch.bfloat16) for L in layers]
    items = lib.matmul_items([it for L, o in zip(layers, outs) for it in L.items(lib, o)])
    ctx.linear_group(items)
    torch.cuda.synchronize()
    first = [t.clone() for o in outs for t in o]
    for o in outs:
        for t in o:
            t.fill_(float("nan"))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ctx.linear_group(items)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.linear_group(items)
    for o in outs:
        for t in o:
            t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(first, [t for o in outs for t in o]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_group_argument_errors(ctx, lib):
    L = Layer(ctx, 256, 768, 768, 400)
    o = L.outputs(torch.bfloat16)
    good = L.items(lib, o)
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_group([])
    assert e.value.status == lib.ERR_SHAPE
    arr = lib.matmul_items(good)
    arr[1].kind = 7
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_group(arr)
    assert e.value.status == lib.ERR_DTYPE
    arr = lib.matmul_items(good)
    arr[2].out = None
    o[0].fill_(float("nan"))
    torch.cuda.synchronize()
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_group(arr)
    assert e.value.status == lib.ERR_NULL
    torch.cuda.synchronize()
    assert torch.isnan(o[0].float()).all()      # a member's error comes back before anything of the group ran
    arr = lib.matmul_items(good)
    arr[2].d_amax_out = o[0].data_ptr()          # the weight-gradient call has no output amax
    with pytest.raises(lib.Fp8Error) as e:
        ctx.linear_group(arr)
    assert e.value.status == lib.ERR_UNSUPPORTED


def test_benchmark_step_in_one_launch(ctx, lib):
    """The twelve matmuls of a c3_llama7b step (8192 tokens) as one fp8_linear_group call, the launch configuration
    bench.py times: every output sampled at 16 positions per 128 x 128 block (and on two whole blocks, first / last
    rows and columns) against the oracle on the oracle's own bytes, and held close to the single calls everywhere."""
    wl = I.WORKLOADS["c3_llama7b"]
    items, per_layer = [], []
    for li, l in enumerate(wl.layers):
        t = I.layer_tensors(wl, li, device="cuda")
        L = Layer(ctx, wl.tokens, l.K, l.N, 0, tensors=(t["x"], t["w"], t["g"]))
        del t
        outs = L.outputs(torch.bfloat16)
        items += L.items(lib, outs)
        per_layer.append((L, outs))
    n0 = lib.launch_count()
    ctx.linear_group(items)
    assert lib.launch_count() - n0 == 1
    torch.cuda.synchronize()
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0
    for li, (L, outs) in enumerate(per_layer):
        single = L.outputs(torch.bfloat16)
        L.single_calls(ctx, single)
        torch.cuda.synchronize()
        for got, one in zip(outs, single):
            assert _close_to_single_call(got, one)
        del single
        rng = np.random.default_rng(li)
        for kind, a8, fa, sa, b8, fb, sb, out in ((O.FWD, L.rx, O.N_E4, L.sx, L.rw, O.N_E4, L.sw, outs[0]),
                                                  (O.DGRAD, L.rg, O.N_E5, L.sg, L.rw, O.N_E4, L.sw, outs[1]),
                                                  (O.WGRAD, L.rg, O.N_E5, L.sg, L.rx, O.N_E4, L.sx, outs[2])):
            rows, cols = tile_sample_positions(rng, out.shape[0], out.shape[1], per_tile=16, full_tiles=2)
            ref = O.linear_samples(kind, a8, fa, sa, b8, fb, sb, rows, cols)
            frac = assert_bf16_within_one_ulp(bits_of(out)[rows, cols], ref)
            print(f"[parity] c3 grouped, layer {li} kind {kind}: {rows.size} positions, {frac:.5f} through the cancellation branch")
