"""Every kernel family, many launches in a row on a GPU kept busy by a second stream: each launch must reproduce the
first one bit for bit.

The kernels hand data between roles through shared memory, tensor memory, barriers and bulk-copy groups; a missing
wait shows only when the timing is unlucky (a staging slab rewritten under a pending store was found this way: zeros
in the last columns of a ragged tile, one launch in twenty, and only with other work in flight).  The first result of
every case is held to the oracle by the parity tests of its own file; here the question is whether launch n gives
the bits of launch 1.  Ragged shapes on purpose: tiles that hang over the edge take the rarely used paths.
"""
import pytest
import torch

from paper_2309_17224_b200 import inputs as I

pytestmark = pytest.mark.gpu

ROUNDS = 60


@pytest.fixture(scope="module")
def lib():
    from paper_2309_17224_b200 import fp8lin
    return fp8lin


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0)
    yield c
    c.close()


class Busy:
    """A second stream that streams a buffer larger than L2 through a copy loop while the block runs."""

    def __init__(self):
        self.stream = torch.cuda.Stream()
        self.a = torch.empty(192 << 20, dtype=torch.uint8, device="cuda")
        self.b = torch.empty_like(self.a)

    def kick(self, n=3):
        with torch.cuda.stream(self.stream):
            for _ in range(n):
                self.b.copy_(self.a)


def _same(first, again):
    return all(torch.equal(a.view(torch.uint8), b.view(torch.uint8)) for a, b in zip(first, again))


def _repeat(ctx, lib, make_outputs, launch, rounds=ROUNDS):
    busy = Busy()
    first = None
    for rnd in range(rounds):
        outs = make_outputs()
        busy.kick()
        launch(outs)
        torch.cuda.synchronize()
        if first is None:
            first = outs
        else:
            assert _same(first, outs), f"launch {rnd} differs from the first"
    assert ctx.device_flags(clear=True) & lib.FLAG_TIMEOUT == 0


def _bytes(T, K, N, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    r8 = lambda r, c: torch.randint(1, 0x78, (r, c), dtype=torch.uint8, device="cuda", generator=g)
    return r8(T, K), r8(N, K), r8(T, N), torch.tensor([3, 2, 9], dtype=torch.int32, device="cuda")


def _nan(shape, dt):
    return torch.full(shape, float("nan"), dtype=dt, device="cuda")


@pytest.mark.parametrize("T,K,N", [(400, 1040, 784), (272, 8208, 304), (528, 272, 144), (2048, 4096, 11008 // 8 * 2)])
@pytest.mark.parametrize("dt", [torch.bfloat16, torch.float32])
def test_matmuls_one_call_each(ctx, lib, T, K, N, dt):
    """CTA-pair kernel (both tile shapes, sliced contraction) on ragged problems: forward, input and weight gradient."""
    x8, w8, g8, b = _bytes(T, K, N, 1)
    amax = torch.zeros(2, dtype=torch.float32, device="cuda")

    def launch(o):
        ctx.linear_fwd(x8, b[1:2], w8, b[0:1], o[0], d_amax_y=amax[0:1])
        ctx.linear_dgrad(g8, b[2:3], w8, None, b[0:1], o[1], d_amax_dx=amax[1:2])
        ctx.linear_wgrad(g8, None, b[2:3], x8, None, b[1:2], o[2], T)
        o.append(amax.clone())

    _repeat(ctx, lib, lambda: [_nan((T, N), dt), _nan((T, K), dt), _nan((N, K), dt)], launch)


@pytest.mark.parametrize("T,K,N", [(1, 8192, 1024), (4, 2064, 784), (16, 4096, 1280), (64, 28672, 512), (128, 1024, 18944)])
def test_decode_matmuls(ctx, lib, T, K, N):
    """Decode kernel: cluster exchange, split through the workspace with the finalize launch, activation quantised in
    the launch, early weight loads."""
    x8, w8, _, b = _bytes(T, K, N, 2)
    x = I.normal_bf16(T, K, 1.0, 7, 1, "cuda", outlier_frac=0.005, outlier_scale=100.0)

    def launch(o):
        ctx.linear_fwd(x8, b[1:2], w8, b[0:1], o[0])
        ctx.linear_infer(x8, b[1:2], w8, b[0:1], o[1])
        ctx.linear_infer_cast(x, o[3], o[4], o[5], w8, b[0:1], o[2])

    _repeat(ctx, lib, lambda: [_nan((T, N), torch.bfloat16), _nan((T, N), torch.bfloat16), _nan((T, N), torch.bfloat16),
                               torch.zeros(1, device="cuda"), torch.full((1,), 77, dtype=torch.int32, device="cuda"),
                               torch.full((T, K), 0x55, dtype=torch.uint8, device="cuda")], launch)


@pytest.mark.parametrize("T,K,N", [(400, 1040, 784), (272, 528, 304)])
def test_fused_epilogues(ctx, lib, T, K, N):
    """GELU forward and backward kinds, with the consumer's FP8 bytes and the amax out of the same launch."""
    x8, w8, g8, b = _bytes(T, K, N, 3)
    bz = torch.tensor([5], dtype=torch.int32, device="cuda")
    pre = I.normal_bf16(T, K, 1.0, 9, 1, "cuda")

    def launch(o):
        ctx.linear_fwd_act(x8, b[1:2], w8, b[0:1], o[0], o[1], d_amax_act=o[6][0:1])
        ctx.linear_fwd_q(x8, b[1:2], w8, b[0:1], o[2], bz, y_pre=o[3], d_amax_z=o[6][1:2], act=lib.ACT_GELU)
        ctx.linear_dgrad_q(g8, b[2:3], w8, None, b[0:1], o[4], bz, y_pre=pre, dx=o[5], d_amax_g=o[6][2:3], act=lib.ACT_GELU)

    _repeat(ctx, lib, lambda: [_nan((T, N), torch.bfloat16), _nan((T, N), torch.bfloat16),
                               torch.full((T, N), 0x55, dtype=torch.uint8, device="cuda"), _nan((T, N), torch.bfloat16),
                               torch.full((T, K), 0x55, dtype=torch.uint8, device="cuda"), _nan((T, K), torch.bfloat16),
                               torch.zeros(3, device="cuda")], launch)
    ctx.device_flags(clear=True)


def test_swiglu_epilogues(ctx, lib):
    T, K, F = 400, 1040, 384          # gate_up has 2F = 768 rows
    x8, w8, _, b = _bytes(T, K, 2 * F, 4)
    dz8 = torch.randint(1, 0x78, (T, K), dtype=torch.uint8, device="cuda")    # a "down" layer's dY: [T, N = K here]
    wd8 = torch.randint(1, 0x78, (K, F), dtype=torch.uint8, device="cuda")    # down weight [N = K, K = F]
    bz = torch.tensor([4], dtype=torch.int32, device="cuda")
    pre = I.normal_bf16(T, 2 * F, 1.0, 11, 1, "cuda")

    def launch(o):
        ctx.linear_fwd_q(x8, b[1:2], w8, b[0:1], o[0], bz, y_pre=o[1], d_amax_z=o[3][0:1], act=lib.ACT_SWIGLU)
        ctx.linear_dgrad_q(dz8, b[2:3], wd8, None, b[0:1], o[2], bz, y_pre=pre, d_amax_g=o[3][1:2], act=lib.ACT_SWIGLU)

    _repeat(ctx, lib, lambda: [torch.full((T, F), 0x55, dtype=torch.uint8, device="cuda"), _nan((T, 2 * F), torch.bfloat16),
                               torch.full((T, 2 * F), 0x55, dtype=torch.uint8, device="cuda"), torch.zeros(2, device="cuda")],
            launch)
    ctx.device_flags(clear=True)


def test_quantisation_calls(ctx, lib):
    """Grouped passes (two-pass and one-pass with wrong guesses), the tile kernel with its transposed copy, the
    decode-size cast and the strided-row amax."""
    shapes = [(400, 1040), (272, 8208), (33, 528), (2048, 4096), (1, 8192)]
    xs = [I.normal_bf16(r, c, 1.0, 13 + i, 1, "cuda", outlier_frac=0.01, outlier_scale=50.0) for i, (r, c) in enumerate(shapes)]

    def make():
        return ([torch.full(s, 0x55, dtype=torch.uint8, device="cuda") for s in shapes] +          # grouped, two passes
                [torch.full(s, 0x55, dtype=torch.uint8, device="cuda") for s in shapes] +          # grouped, one pass
                [torch.full(s, 0x55, dtype=torch.uint8, device="cuda") for s in shapes] +          # per tensor, with y_t
                [torch.full((c, r), 0x55, dtype=torch.uint8, device="cuda") for r, c in shapes] +
                [torch.zeros((3, len(shapes)), device="cuda"), torch.full((3, len(shapes)), 40, dtype=torch.int32, device="cuda")])

    def launch(o):
        n = len(shapes)
        am, bi = o[4 * n], o[4 * n + 1]
        ctx.cast_group([(lib.E4, x, am[0, i:i + 1], bi[0, i:i + 1], o[i]) for i, x in enumerate(xs)])
        ctx.cast_group([(lib.E5, x, am[1, i:i + 1], bi[1, i:i + 1], o[n + i]) for i, x in enumerate(xs)], predicted=True)
        for i, x in enumerate(xs):
            y_t = o[3 * n + i] if x.shape[0] % 16 == 0 else None   # the transposed copy's rows are 16-byte multiples
            ctx.cast_e4(x, None, d_amax_out=am[2, i:i + 1], d_bias_out=bi[2, i:i + 1], y=o[2 * n + i], y_t=y_t)

    _repeat(ctx, lib, make, launch, rounds=30)
    ctx.device_flags(clear=True)
    ctx.prediction_stats(clear=True)


def test_fp16_accumulation_kind(ctx, lib):
    T, K, N = 272, 1040, 528
    x8, w8, _, b = _bytes(T, K, N, 5)
    b = torch.tensor([-2, -3, 0], dtype=torch.int32, device="cuda")   # small scaled values: the FP16 sums stay finite

    def launch(o):
        ctx.linear_f16acc(0, x8, b[1:2], w8, b[0:1], o[0], T, K, N, chunk=256)

    _repeat(ctx, lib, lambda: [_nan((T, N), torch.float16)], launch, rounds=30)
