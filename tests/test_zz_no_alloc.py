"""unipool_dispatch_static - the token permute for embedders that may not allocate device memory
(a memory-planned runtime, a plugin that only sees one call's tensors) and so cannot provide the
context's workspace.  Its scratch is an array inside the library.  The result must be the one
unipool_dispatch gives, bit for bit, also on the second call, when the array still holds the
first call's histograms."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_dispatch_static_matches_dispatch_twice_in_a_row(dtype):
    import torch
    from paper_2605_06665_b200 import binding as B
    from paper_2605_06665_b200 import build as builder
    builder.build()
    d, f, k, M_pool = 256, 128, 2, 96
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    code = B.BF16 if dtype == "bf16" else B.FP32
    T_max = 3000
    cfg = B.make_config(d, f, M_pool, k, 1, T_max, code, 1e-6, 2.0)
    ctx = B.Context(cfg, "cuda")
    cap = ctx.row_capacity
    g = torch.Generator(device="cpu").manual_seed(7)
    i32 = torch.int32

    def outputs():
        return dict(offsets=torch.full((M_pool + 1,), -7, dtype=i32, device="cuda"),
                    row_of=torch.full((T_max, k), -7, dtype=i32, device="cuda"),
                    token_of=torch.full((cap,), -7, dtype=i32, device="cuda"),
                    tile_expert=torch.full((cap // B.ROW_ALIGN,), -7, dtype=i32, device="cuda"),
                    Xp=torch.full((cap, d), 3.0, dtype=tdt, device="cuda"))

    # two calls in a row on different batches: the second meets the first one's leftovers
    for T, M in ((3000, 96), (1234, 40)):
        x = torch.randn(T, d, generator=g).to(tdt).cuda()
        scores = torch.rand(T, M, generator=g)
        idx = scores.topk(k, dim=1).indices.to(i32).cuda()
        ref, got = outputs(), outputs()
        ctx.dispatch(x, T, idx, M, ref["offsets"], ref["row_of"], ref["token_of"], ref["tile_expert"], ref["Xp"])
        B.dispatch_static(x, T, d, code, k, idx, M, cap, got["offsets"], got["row_of"], got["token_of"],
                          got["tile_expert"], got["Xp"])
        torch.cuda.synchronize()
        used = int(ref["offsets"][M])
        assert used >= T * k
        assert torch.equal(got["offsets"][:M + 1], ref["offsets"][:M + 1])
        assert torch.equal(got["row_of"][:T], ref["row_of"][:T])
        assert torch.equal(got["token_of"], ref["token_of"])
        assert torch.equal(got["tile_expert"], ref["tile_expert"])
        assert torch.equal(got["Xp"][:used].view(torch.uint8), ref["Xp"][:used].view(torch.uint8))
        # and it is the permutation: every row holds its token, pad rows are zero
        tok = got["token_of"][:used].cpu().numpy()
        Xp = got["Xp"][:used].float().cpu().numpy()
        xs = x.float().cpu().numpy()
        assert (Xp[tok >= 0] == xs[tok[tok >= 0]]).all() and not Xp[tok < 0].any()
    ctx.check_status()
    ctx.close()


def test_dispatch_static_refuses_what_does_not_fit():
    import torch
    from paper_2605_06665_b200 import binding as B
    d, k, M = 64, 1, 512
    T = 270000                                   # ceil(T/256) * 512 entries > the built-in scratch
    cap = (T * k + M * 127 + 127) // 128 * 128
    one = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.UniPoolError) as ei:
        B.dispatch_static(one, T, d, B.FP32, k, one, M, cap, one, one, one, one, one)
    assert ei.value.code == -3 and "scratch" in str(ei.value)


def test_dispatch_static_without_tokens_and_with_a_bad_index():
    """Two corners of the entry point: T = 0 leaves empty maps, and an expert id outside the router's
    range is dropped (row_of = -1; there is no status word to report it through) while every other
    assignment keeps the row the reference call gives it."""
    import torch
    from paper_2605_06665_b200 import binding as B
    d, f, k, M = 128, 128, 2, 16
    T = 700
    cfg = B.make_config(d, f, M, k, 1, T, B.FP32, 1e-6, 2.0)
    ctx = B.Context(cfg, "cuda")
    cap = ctx.row_capacity
    i32 = torch.int32
    g = torch.Generator(device="cpu").manual_seed(11)
    x = torch.randn(T, d, generator=g).cuda()
    idx = torch.rand(T, M, generator=g).topk(k, dim=1).indices.to(i32).cuda()

    def outputs():
        return dict(offsets=torch.full((M + 1,), -7, dtype=i32, device="cuda"),
                    row_of=torch.full((T, k), -7, dtype=i32, device="cuda"),
                    token_of=torch.full((cap,), -7, dtype=i32, device="cuda"),
                    tile_expert=torch.full((cap // B.ROW_ALIGN,), -7, dtype=i32, device="cuda"),
                    Xp=torch.zeros(cap, d, device="cuda"))

    o = outputs()
    B.dispatch_static(x, 0, d, B.FP32, k, idx, M, cap, o["offsets"], o["row_of"], o["token_of"], o["tile_expert"], o["Xp"])
    torch.cuda.synchronize()
    assert not o["offsets"].any() and (o["token_of"] == -1).all() and (o["tile_expert"] == -1).all()

    bad = idx.clone()
    bad[5, 1] = M + 3                                        # out of range: dropped
    ref, got = outputs(), outputs()
    ctx.dispatch(x, T, bad, M, ref["offsets"], ref["row_of"], ref["token_of"], ref["tile_expert"], ref["Xp"])
    B.dispatch_static(x, T, d, B.FP32, k, bad, M, cap, got["offsets"], got["row_of"], got["token_of"],
                      got["tile_expert"], got["Xp"])
    torch.cuda.synchronize()
    with pytest.raises(B.UniPoolError):                      # the context's call reports it ...
        ctx.check_status()
    assert int(got["row_of"][5, 1]) == -1                    # ... the static one can only drop it
    assert torch.equal(got["row_of"], ref["row_of"]) and torch.equal(got["offsets"], ref["offsets"])
    assert torch.equal(got["token_of"], ref["token_of"])
    assert int(got["offsets"][M]) >= T * k - 1
    ctx.close()

