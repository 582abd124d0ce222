"""The no-allocation amax entry point against the regular one.

Some users of the library cannot let it allocate: they gave all device memory
to their own pool at start-up, or they may not call cudaMalloc on the thread
that serves requests.  ``fp8_amax_noalloc`` is for them: no context, no
allocation, a fixed workspace inside the library.  This file checks, through
the C ABI, that it returns exactly what ``fp8_amax`` returns, on two calls in a
row (the second must not see anything the first left in the shared workspace).
It sorts last on purpose, so that a run that stops at the first failure has
already been through every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _amax_pair(lib, ctx, x):
    want = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    got = torch.full((1,), -2.0, dtype=torch.float32, device="cuda")
    ctx.amax(x, want)
    lib.amax_noalloc(x, got)
    return float(got.item()), float(want.item())


def test_noalloc_amax_matches_the_regular_entry_point_twice_in_a_row():
    from paper_2309_17224_b200 import fp8lin as lib
    ctx = lib.Context(0)
    g = torch.Generator(device="cuda").manual_seed(2309)
    big = (torch.randn((1031, 4099), generator=g, device="cuda") * 40.0).to(torch.bfloat16)   # many chunks, ragged tail
    small = (torch.randn((300, 520), generator=g, device="cuda") * 0.01).to(torch.bfloat16)   # much smaller amax
    # two calls in a row: the large maximum of the first must not leak into the second
    got1, want1 = _amax_pair(lib, ctx, big)
    got2, want2 = _amax_pair(lib, ctx, small)
    assert got1 == want1 and got1 == float(big.float().abs().max().item())
    assert got2 == want2 and got2 == float(small.float().abs().max().item())
    # and again in the other order, back to back on the stream with no host sync in between
    outs = torch.zeros(4, dtype=torch.float32, device="cuda")
    lib.amax_noalloc(small, outs[0:1])
    lib.amax_noalloc(big, outs[1:2])
    lib.amax_noalloc(small, outs[2:3])
    tiny = big[:1, :5].clone()   # fewer elements than one 16-byte vector
    lib.amax_noalloc(tiny, outs[3:4])
    assert outs.tolist() == [want2, want1, want2, float(tiny.float().abs().max().item())]
    # special values behave like the regular entry point
    big[500, 77] = float("inf")
    got, want = _amax_pair(lib, ctx, big)
    assert got == want == float("inf")
    big[3, 3] = float("nan")
    got, want = _amax_pair(lib, ctx, big)
    assert np.isnan(got) and np.isnan(want)
    ctx.close()


def test_noalloc_amax_rejects_what_it_cannot_do():
    from paper_2309_17224_b200 import fp8lin as lib
    x = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    with pytest.raises(lib.Fp8Error) as e:     # beyond the fixed workspace: 2^29 elements
        lib.amax_noalloc(x, out, rows=1 << 20, cols=1 << 10, ld=1 << 10)
    assert e.value.status == lib.ERR_TOO_LARGE
    with pytest.raises(lib.Fp8Error) as e:     # strided rows are not supported here
        lib.amax_noalloc(x, out, rows=64, cols=32, ld=64)
    assert e.value.status == lib.ERR_UNSUPPORTED
    with pytest.raises(lib.Fp8Error) as e:
        lib.amax_noalloc(x.view(-1)[1:129].view(1, 128), out)
    assert e.value.status == lib.ERR_ALIGN
