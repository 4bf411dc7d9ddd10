"""GPU parity: every step of the CUDA path against the CPU oracle on the same
seeded inputs, through the C-ABI (ctypes) binding.

Tolerances (max|gpu - ref| / max|ref|): 1e-5 in fp32 mode, 1e-2 for bf16 storage
with fp32 accumulation; balance loss relative 1e-5; routing indices, counts and
the permutation maps bit-exact (indices: where the logit margin exceeds 1e-4).
"""
import os

import numpy as np
import pytest

from oracle import unipool_oracle as O
from paper_2605_06665_b200 import synth
from parity_utils import (MARGIN, build_stack, calib_c, check_routing, f64, margin_safe, oracle_params,
                          rel_max, to_np)

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-5, "bf16": 1e-2}


def small_cfg(**kw):
    cfg = dict(L=2, d=128, f=192, M=8, k=2, T=300, dtype="fp32", private=0, zipf_beta=0.0)
    cfg.update(kw)
    return cfg


def run_layer_checks(cfg, T, L, seed=0, zero_grad_check=True):
    """Runs the stack layer by layer; each layer's oracle consumes the GPU's own
    x_l (and dx_{l+1}) so that only this layer's arithmetic is compared."""
    import torch
    inputs = synth.make_inputs(cfg, seed=seed, T=T, L=L)
    st = build_stack(cfg, inputs, T=T, L=L)
    tol = TOL[cfg["dtype"]]
    k, m, M = cfg["k"], synth.router_width(cfg), cfg["M"]
    mode = cfg.get("router", "norm")
    pool, routers = oracle_params(inputs, L, mode)
    c, eps, alpha = st.c, synth.EPS, synth.ALPHA
    st.x[0].copy_(torch.from_numpy(inputs["x0"]))
    caches = []
    for l in range(L):
        st.forward_layer(l)
        torch.cuda.synchronize()
        x_l = f64(to_np(st.x[l]))
        ref = O.route(x_l, routers[l]["W_r"], routers[l]["sigma"], c, eps, k, routers[l]["bias"], mode=mode)
        idx_gpu = to_np(st.idx[l])
        set_safe, order_safe = check_routing(idx_gpu, ref["z"], ref["idx"], k, mode)
        assert rel_max(to_np(st.z[l]), ref["z"]) < 1e-5
        assert rel_max(to_np(st.znorm[l]), ref["n"]) < 1e-5
        # everything downstream is compared with the GPU's own (valid) routing decision
        ref = O.route(x_l, routers[l]["W_r"], routers[l]["sigma"], c, eps, k, routers[l]["bias"], forced_idx=idx_gpu,
                      mode=mode)
        assert rel_max(to_np(st.gate[l]), ref["g"]) < 1e-5
        assert (to_np(st.counts[l]) == ref["counts"]).all()
        assert to_np(st.counts[l]).sum() == T * k
        assert rel_max(to_np(st.score_sum[l]), ref["S"]) < 1e-5
        # permutation maps: bit-exact
        off, row_of, token_of = O.dispatch_map(idx_gpu, m, 128)
        assert (to_np(st.offsets[l]) == off).all()
        assert (to_np(st.row_of[l]) == row_of).all()
        used = int(off[-1])
        tok_gpu = to_np(st.token_of[l])
        assert (tok_gpu[:used] == token_of).all() and (tok_gpu[used:] == -1).all()
        te = to_np(st.tile_expert[l])
        exp_te = np.full(te.shape, -1)
        for e in range(m):
            exp_te[off[e] // 128:off[e + 1] // 128] = e
        assert (te == exp_te).all()
        Xp = to_np(st.Xp[l])[:used]
        x_gpu = to_np(st.x[l])
        assert (Xp[token_of >= 0] == x_gpu[token_of[token_of >= 0]]).all()      # pure data movement
        assert not Xp[token_of < 0].any()
        # expert FFN on the permuted rows
        base = synth.expert_base(cfg, l)
        GU, A, Yp = to_np(st.GU[l])[:used], to_np(st.A[l])[:used], to_np(st.Yp[l])[:used]
        G_ref, U_ref, A_ref, Y_ref = (np.zeros((used, cfg["f"])), np.zeros((used, cfg["f"])),
                                      np.zeros((used, cfg["f"])), np.zeros((used, cfg["d"])))
        for e in range(m):
            r0, r1 = int(off[e]), int(off[e + 1])
            if r1 > r0:
                G_ref[r0:r1], U_ref[r0:r1], A_ref[r0:r1], Y_ref[r0:r1] = O.expert_ffn(
                    f64(Xp[r0:r1]), pool["W_gate"][base + e], pool["W_up"][base + e], pool["W_down"][base + e])
        assert rel_max(GU[:, :cfg["f"]], G_ref) < tol and rel_max(GU[:, cfg["f"]:], U_ref) < tol
        assert rel_max(A, A_ref) < tol and rel_max(Yp, Y_ref) < tol
        assert not GU[token_of < 0].any() and not Yp[token_of < 0].any()        # pad rows stay zero
        y_ref = O.moe_layer_output(x_l, idx_gpu, ref["g"], pool, base)
        assert rel_max(to_np(st.x[l + 1]), x_l + y_ref) < tol
        ref["x"] = x_l
        caches.append(ref)
    # balance loss
    st.aux_loss()
    torch.cuda.synchronize()
    counts = np.stack([cc["counts"] for cc in caches])
    S = np.stack([f64(to_np(st.score_sum[l])) for l in range(L)])
    if cfg["private"]:
        coefs = []
        for l in range(L):
            lo, fb, co = O.pool_aux_loss(counts[l:l + 1], S[l:l + 1], T, k, alpha)
            assert abs(float(st.loss[l]) - lo) <= 1e-5 * abs(lo)
            assert rel_max(to_np(st.coef[l]), co) < 1e-5
            coefs.append(co)
    else:
        lo, fb, co = O.pool_aux_loss(counts, S, T, k, alpha)
        assert abs(float(st.loss[0]) - lo) <= 1e-5 * abs(lo)
        assert rel_max(to_np(st.coef[0]), co) < 1e-5 and rel_max(to_np(st.fbar[0]), fb) < 1e-5
        coefs = [co] * L
    # backward, layer by layer
    st.zero_grad()
    pool_grad = O.zeros_like_pool(pool)
    dx_cur = torch.from_numpy(inputs["upstream"]).to(st.device, st.tdtype)
    for l in reversed(range(L)):
        dx_out = torch.empty_like(dx_cur)
        st.backward_layer(l, dx_cur, dx_out)
        torch.cuda.synchronize()
        cc = caches[l]
        base = synth.expert_base(cfg, l)
        dxn = f64(to_np(dx_cur))
        dx_e, dg = O.expert_path_backward(cc["x"], cc["idx"], cc["g"], pool, dxn, base, pool_grad)
        assert rel_max(to_np(st.dgate), dg) < tol
        rb = O.route_backward(cc["x"], routers[l]["W_r"], routers[l]["sigma"], c, eps, cc["z"], cc["n"],
                              cc["idx"], dg, coefs[l], mode=mode)
        assert rel_max(to_np(dx_out), dxn + dx_e + rb["dx"]) < tol
        assert rel_max(to_np(st.dW_r[l]), rb["dW_r"]) < tol
        if cfg["dtype"] == "fp32":
            assert abs(float(st.dsigma[l]) - rb["dsigma"]) <= tol * max(abs(rb["dsigma"]), 1e-3)
        else:
            # dsigma is a signed sum over all (token, expert) terms whose inputs (dgate) carry bf16
            # rounding: the bound scales with the sum of their magnitudes, not with the (cancelling) total
            ne = cc["n"] + eps
            dsigma_scale = c * np.sum(np.abs(rb["ds"]) * np.maximum(cc["z"], 0.0) / ne[:, None])
            assert abs(float(st.dsigma[l]) - rb["dsigma"]) <= tol * max(dsigma_scale, 1e-3)
        dx_cur = dx_out
    f = cfg["f"]
    dW_gu = to_np(st.dW_gu)
    assert rel_max(dW_gu[:, :f], pool_grad["W_gate"]) < tol
    assert rel_max(dW_gu[:, f:], pool_grad["W_up"]) < tol
    assert rel_max(to_np(st.dW_down), pool_grad["W_down"]) < tol
    if zero_grad_check:
        used_experts = np.unique(np.concatenate(
            [synth.expert_base(cfg, l) + cc["idx"].reshape(-1) for l, cc in enumerate(caches)]))
        unused = np.setdiff1d(np.arange(M), used_experts)
        assert not dW_gu[unused].any() and not to_np(st.dW_down)[unused].any()
    st.ctx.check_status()
    st.close()


def test_tiny_fp32_layers():
    cfg = synth.CONFIGS["tiny_fp32"]
    run_layer_checks(cfg, cfg["T"], cfg["L"])


@pytest.mark.parametrize("kw,T", [
    (dict(), 300),                                   # ragged T, two tiles per group at most
    (dict(M=5, k=1), 77),                            # k = 1, M not a multiple of anything
    (dict(M=40, k=8, d=64, f=64), 130),              # k = 8
    (dict(M=12, k=2, private=4, L=3), 200),          # layer-private layout (Eq. 1)
    (dict(M=33, k=3), 1),                            # a single token: most experts empty
    (dict(M=8, k=2, zipf_beta=3.0), 700),            # one giant group, several empty experts
    (dict(M=512, k=8, d=64, f=64), 40),              # the largest pool and top-k, the smallest widths
])
def test_small_fp32_shapes(kw, T):
    cfg = small_cfg(**kw)
    run_layer_checks(cfg, T, cfg["L"], seed=3)


@pytest.mark.parametrize("kw,T", [
    (dict(dtype="bf16", d=256, f=384, M=16, k=2), 1000),
    (dict(dtype="bf16", d=128, f=128, M=384, k=8, zipf_beta=0.4), 600),
    (dict(dtype="bf16", d=256, f=256, M=12, k=2, private=4, L=3), 520),
    (dict(dtype="bf16", d=128, f=128, M=10, k=3), 333),     # logit rows that are not 16-byte aligned
    (dict(dtype="bf16", d=64, f=64, M=512, k=8), 257),      # the largest pool and top-k, the smallest widths
    (dict(dtype="bf16", d=128, f=192, M=16, k=2), 1),       # a single token
    # groups of several row tiles: the four row-tile GEMMs run on CTA pairs
    (dict(dtype="bf16", d=256, f=320, M=4, k=2, zipf_beta=1.0), 2100),   # skewed: odd and even tile counts, f % 128 = 64
    (dict(dtype="bf16", d=192, f=256, M=2, k=1), 2500),                  # d % 256 = 192: a clipped last column tile
    (dict(dtype="bf16", d=256, f=256, M=6, k=2, private=2, L=3), 1100),  # private experts through pool views
])
def test_small_bf16_shapes(kw, T):
    cfg = small_cfg(**kw)
    run_layer_checks(cfg, T, cfg["L"], seed=4)


@pytest.mark.parametrize("kw,T", [
    (dict(router="softmax"), 300),                                            # fp32, shared pool, top-2
    (dict(router="softmax", M=24, k=1, private=8, L=3), 260),                 # the paper's baseline: private experts, top-1
    (dict(router="softmax", M=33, k=3, zipf_beta=2.0), 150),                  # skewed logits, ragged width
    (dict(router="softmax", dtype="bf16", d=256, f=256, M=96, k=2), 700),     # tensor-core router
    (dict(router="softmax", dtype="bf16", d=128, f=128, M=10, k=1), 333),     # unaligned logit rows
    (dict(router="softmax", dtype="bf16", d=128, f=128, M=384, k=8, zipf_beta=0.4), 400),
    (dict(router="softmax", dtype="bf16", d=256, f=256, M=24, k=1, private=8, L=3), 520),
])
def test_softmax_router_mode(kw, T):
    """The conventional softmax router (the baselines of Sec. 5.1, the ablation rows of Sec. 5.3)
    through the same calls: probabilities as scores and gates, the same selection, statistics and
    balance loss, and its own derivative."""
    cfg = small_cfg(**kw)
    run_layer_checks(cfg, T, cfg["L"], seed=6)


def test_tiny_fp32_end_to_end():
    """Config 1 without teacher forcing: forward, balance loss and backward of the
    whole 4-layer stack against the float64 oracle."""
    import torch
    cfg = synth.CONFIGS["tiny_fp32"]
    inputs = synth.make_inputs(cfg, seed=0)
    st = build_stack(cfg, inputs)
    L, T, k = cfg["L"], cfg["T"], cfg["k"]
    pool, routers = oracle_params(inputs, L)
    x0 = torch.from_numpy(inputs["x0"]).cuda()
    up = torch.from_numpy(inputs["upstream"]).cuda()
    st.zero_grad()
    dx0 = st.step(x0, up)
    torch.cuda.synchronize()
    idx_gpu = [to_np(st.idx[l]) for l in range(L)]
    free = O.stack_forward(f64(inputs["x0"]), routers, pool, k, st.c, synth.EPS)
    for l in range(L):
        check_routing(idx_gpu[l], free[l]["z"], free[l]["idx"], k)
    res = O.stack_objective_and_grads(f64(inputs["x0"]), routers, pool, k, st.c, synth.EPS, synth.ALPHA,
                                      f64(inputs["upstream"]), forced_idx=idx_gpu)
    assert rel_max(to_np(st.x[L]), res["caches"][-1]["x_next"]) < 1e-5
    assert abs(float(st.loss[0]) - res["loss_aux"]) <= 1e-5 * abs(res["loss_aux"])
    f = cfg["f"]
    assert rel_max(to_np(st.dW_gu)[:, :f], res["pool_grad"]["W_gate"]) < 1e-5
    assert rel_max(to_np(st.dW_gu)[:, f:], res["pool_grad"]["W_up"]) < 1e-5
    assert rel_max(to_np(st.dW_down), res["pool_grad"]["W_down"]) < 1e-5
    for l in range(L):
        assert rel_max(to_np(st.dW_r[l]), res["router_grads"][l]["dW_r"]) < 1e-5
        assert abs(float(st.dsigma[l]) - res["router_grads"][l]["dsigma"]) <= 1e-5 * max(
            1e-3, abs(res["router_grads"][l]["dsigma"]))
    assert rel_max(to_np(dx0), res["dx0"]) < 1e-5
    # determinism: a second pass gives bit-identical outputs and twice the gradients
    xL_1 = st.x[L].clone()
    g1 = st.dW_down.clone()
    st.step(x0, up)
    torch.cuda.synchronize()
    assert torch.equal(xL_1, st.x[L])
    assert rel_max(to_np(st.dW_down), 2 * to_np(g1)) < 1e-6
    # a pass that overwrites needs no zeroed buffers: start from garbage, end at one pass's gradient
    st.dW_gu.fill_(7.0); st.dW_down.fill_(-3.0); st.dW_r.fill_(5.0)
    st.step(x0, up, accumulate=False)
    torch.cuda.synchronize()
    assert rel_max(to_np(st.dW_down), to_np(g1)) < 1e-6
    assert rel_max(to_np(st.dW_gu)[:, :f], res["pool_grad"]["W_gate"]) < 1e-5
    st.close()


def test_fp32_router_weights_in_bf16_mode():
    """Router weights are fp32 numbers even when activations are bf16: the tensor-core logits
    (weights split into three bf16 terms) must still be the fp32 logits of the unrounded weights."""
    import torch
    cfg = small_cfg(dtype="bf16", d=256, f=128, M=40, k=2, L=1)
    T = 700
    inputs = synth.make_inputs(cfg, seed=8, T=T)
    rng = np.random.default_rng(11)
    W = (inputs["routers"][0]["W_r"] * (1.0 + 1e-3 * rng.standard_normal((40, 256)))).astype(np.float32)
    assert (synth.round_to_bf16(W) != W).any()
    inputs["routers"][0]["W_r"] = W
    st = build_stack(cfg, inputs, T=T)
    st.x[0].copy_(torch.from_numpy(inputs["x0"]))
    st.forward_layer(0)
    torch.cuda.synchronize()
    ref = O.route(f64(inputs["x0"]), f64(W), 1.0, st.c, synth.EPS, 2)
    assert rel_max(to_np(st.z[0]), ref["z"]) < 1e-5
    check_routing(to_np(st.idx[0]), ref["z"], ref["idx"], 2)
    ref = O.route(f64(inputs["x0"]), f64(W), 1.0, st.c, synth.EPS, 2, forced_idx=to_np(st.idx[0]))
    assert rel_max(to_np(st.gate[0]), ref["g"]) < 1e-5
    assert rel_max(to_np(st.score_sum[0]), ref["S"]) < 1e-5
    st.ctx.check_status()
    st.close()


def test_cuda_graph_replay_matches_eager_step():
    """A step recorded into a CUDA graph issues the same kernels: replaying it reproduces the eager
    step's outputs and gradients bit for bit (overwriting pass, deterministic kernels)."""
    import torch
    cfg = small_cfg(dtype="bf16", d=256, f=384, M=16, k=2, L=3)
    T = 900
    inputs = synth.make_inputs(cfg, seed=9, T=T)
    x0 = torch.from_numpy(inputs["x0"]).cuda().bfloat16()
    up = torch.from_numpy(inputs["upstream"]).cuda().bfloat16()
    st = build_stack(cfg, inputs, T=T, deferred_wgrad=True)
    st.step(x0, up, accumulate=False)
    torch.cuda.synchronize()
    ref = [t.clone() for t in (st.x[cfg["L"]], st.dW_gu, st.dW_down, st.dW_r, st.loss, st.idx)]
    graph = st.capture_step(x0, up, accumulate=False)
    for t in (st.x, st.dW_gu, st.dW_down, st.dW_r):
        t.fill_(1.0)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    st.ctx.check_status()
    got = (st.x[cfg["L"]], st.dW_gu, st.dW_down, st.dW_r, st.loss, st.idx)
    for a, b in zip(ref[:3] + ref[5:], got[:3] + got[5:]):
        assert torch.equal(a, b)
    assert rel_max(to_np(got[3]), to_np(ref[3])) < 1e-5             # fp32 add-reduce order may differ
    assert torch.allclose(ref[4], got[4], rtol=1e-6)
    st.close()


def test_single_replica_exchange_step_is_the_plain_step():
    """The data-parallel step with one replica (every collective is the identity) issues the weight
    gradient as two single-product passes: same outputs and gradients as the plain step."""
    import torch
    from paper_2605_06665_b200 import dp
    cfg = small_cfg(dtype="bf16", d=256, f=384, M=16, k=2, L=4, groups=2)
    T = 700
    inputs = synth.make_inputs(cfg, seed=10, T=T)
    x0 = torch.from_numpy(inputs["x0"]).cuda().bfloat16()
    up = torch.from_numpy(inputs["upstream"]).cuda().bfloat16()
    for deferred in (True, False):
        st = build_stack(cfg, inputs, T=T, deferred_wgrad=deferred)
        st.step(x0, up, accumulate=False)
        torch.cuda.synchronize()
        ref = [t.clone() for t in (st.x[cfg["L"]], st.dW_gu, st.dW_down, st.loss, st.dW_r)]
        for t in (st.dW_gu, st.dW_down):
            t.fill_(1.0)                               # an overwriting step leaves nothing of this behind
        st.step(x0, up, accumulate=False, exchange=dp.GradientExchange(1))
        torch.cuda.synchronize()
        st.ctx.check_status()
        got = (st.x[cfg["L"]], st.dW_gu, st.dW_down, st.loss, st.dW_r)
        for a, b in zip(ref[:4], got[:4]):
            assert torch.equal(a, b)
        assert rel_max(to_np(got[4]), to_np(ref[4])) < 1e-5
        st.close()


def test_microbatches_with_single_replica_exchange():
    """Micro-batch accumulation through the data-parallel exchange with one replica (every collective
    the identity) reproduces the plain accumulation: losses and f-bar bit for bit, the gradients up to
    the order of the fp32 add-reduces of the later micro-batches."""
    import torch
    from paper_2605_06665_b200 import dp
    cfg = small_cfg(dtype="bf16", d=256, f=384, M=16, k=2, L=3)
    T = 500
    batches = []
    for seed in (20, 21, 22):
        inp = synth.make_inputs(cfg, seed=seed, T=T)
        batches.append((torch.from_numpy(inp["x0"]).cuda().bfloat16(), torch.from_numpy(inp["upstream"]).cuda().bfloat16()))
    inputs = synth.make_inputs(cfg, seed=20, T=T)
    results = []
    for exchange in (None, dp.GradientExchange(1)):
        st = build_stack(cfg, inputs, T=T, deferred_wgrad=True)
        losses = st.accumulate_microbatches(batches, exchange=exchange)
        torch.cuda.synchronize()
        st.ctx.check_status()
        results.append([t.clone() for t in (st.dW_gu, st.dW_down, st.dW_r, st.fbar_lag, torch.stack(losses))])
        st.close()
    for a, b in zip(results[0][:3], results[1][:3]):
        assert rel_max(to_np(b), to_np(a)) < 1e-6
    for a, b in zip(results[0][3:], results[1][3:]):
        assert torch.equal(a, b)


def test_host_resident_step_matches_device_resident_step():
    """Inputs in pinned host memory (upstream copied in during the forward pass, x_L copied out during
    the backward pass, on a second stream) give the same step, eagerly and from a CUDA graph."""
    import torch
    cfg = small_cfg(dtype="bf16", d=256, f=384, M=16, k=2, L=3)
    T = 900
    inputs = synth.make_inputs(cfg, seed=12, T=T)
    x0_h = torch.from_numpy(inputs["x0"]).bfloat16().pin_memory()
    up_h = torch.from_numpy(inputs["upstream"]).bfloat16().pin_memory()
    out_h = torch.zeros_like(x0_h).pin_memory()
    st = build_stack(cfg, inputs, T=T, deferred_wgrad=True)
    dx_ref = st.step(x0_h.cuda(), up_h.cuda(), accumulate=False).clone()
    torch.cuda.synchronize()
    ref = [t.clone() for t in (st.x[cfg["L"]], st.dW_gu, st.dW_down)]
    for eager in (True, False):
        for t in (st.x, st.dW_gu, st.dW_down, st.dx):
            t.fill_(1.0)
        out_h.zero_()
        if eager:
            dx = st.step(x0_h, up_h, accumulate=False, out=out_h)
        else:
            graph = st.capture_step(x0_h, up_h, accumulate=False, out=out_h)
            out_h.zero_()
            st.dx.fill_(1.0)
            graph.replay()
            dx = st.dx[cfg["L"] % 2]
        torch.cuda.synchronize()
        st.ctx.check_status()
        assert torch.equal(st.x[cfg["L"]], ref[0]) and torch.equal(out_h.cuda(), ref[0])
        assert torch.equal(st.dW_gu, ref[1]) and torch.equal(st.dW_down, ref[2])
        assert torch.equal(dx, dx_ref)
    st.close()


def test_empty_batch():
    import torch
    cfg = small_cfg()
    inputs = synth.make_inputs(cfg, seed=1)
    st = build_stack(cfg, inputs)
    st.counts.fill_(7)
    st.offsets.fill_(7)
    st.zero_grad()
    st.forward(T=0)
    st.aux_loss(T=1)
    st.backward(T=0)
    torch.cuda.synchronize()
    assert not to_np(st.counts).any() and not to_np(st.offsets).any()
    assert not to_np(st.dW_gu).any()
    st.ctx.check_status()
    st.close()


@pytest.mark.parametrize("kw,T", [
    (dict(dtype="bf16", d=256, f=384, M=16, k=2, L=3), 900),
    (dict(dtype="bf16", d=128, f=64, M=64, k=2, L=2, zipf_beta=0.5), 200),     # experts without any row
    (dict(dtype="fp32", d=128, f=192, M=24, k=2, L=2, zipf_beta=0.5), 150),
])
def test_deferred_pool_wgrad_matches_per_layer_accumulation(kw, T):
    """Weight gradients contracted over all layers at once, and passes that overwrite the
    pool-gradient buffers instead of adding to them, give the per-layer accumulation's result."""
    import torch
    cfg = small_cfg(**kw)
    inputs = synth.make_inputs(cfg, seed=5, T=T)
    tdt = torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32
    x0 = torch.from_numpy(inputs["x0"]).cuda().to(tdt)
    up = torch.from_numpy(inputs["upstream"]).cuda().to(tdt)
    grads = []
    for deferred, accumulate in ((False, True), (True, True), (False, False), (True, False)):
        st = build_stack(cfg, inputs, T=T, deferred_wgrad=deferred)
        if accumulate:
            st.zero_grad()
        else:                          # overwriting passes start from garbage
            st.dW_gu.fill_(11.0); st.dW_down.fill_(-2.0)
        st.step(x0, up, accumulate=accumulate)
        torch.cuda.synchronize()
        st.ctx.check_status()
        grads.append((to_np(st.dW_gu), to_np(st.dW_down)))
        st.close()
    assert np.abs(grads[0][0]).max() > 0
    for g in grads[1:]:
        assert rel_max(g[0], grads[0][0]) < 1e-5
        assert rel_max(g[1], grads[0][1]) < 1e-5


def test_one_step_behind_fbar():
    import torch
    cfg = small_cfg(M=8)
    inputs = synth.make_inputs(cfg, seed=6)
    st = build_stack(cfg, inputs)
    st.forward(torch.from_numpy(inputs["x0"]).cuda())
    prev = np.random.default_rng(0).dirichlet(np.ones(8)).astype(np.float32)
    st.aux_loss(fbar_prev=torch.from_numpy(prev).cuda())
    torch.cuda.synchronize()
    lo, fb, co = O.pool_aux_loss(to_np(st.counts).astype(np.int64), f64(to_np(st.score_sum)), cfg["T"], cfg["k"],
                                 synth.ALPHA, fbar_prev=f64(prev))
    assert abs(float(st.loss[0]) - lo) <= 1e-5 * abs(lo)
    assert rel_max(to_np(st.coef[0]), co) < 1e-5 and rel_max(to_np(st.fbar[0]), fb) < 1e-5
    st.close()


def test_microbatches_accumulate_with_one_step_behind_fbar():
    """App. G: three micro-batches add into the same gradient buffers; the balance loss of each uses
    the token fractions of the one before (uniform for the first).  Against the float64 oracle run
    micro-batch by micro-batch with the same lagged f-bar."""
    import torch
    cfg = synth.CONFIGS["tiny_fp32"]
    L, T, k, M = cfg["L"], cfg["T"], cfg["k"], cfg["M"]
    base = synth.make_inputs(cfg, seed=0)
    pool, routers = oracle_params(base, L)
    st = build_stack(cfg, base)
    batches, idxs = [], []
    for i in range(3):
        inp = synth.make_inputs(cfg, seed=20 + i)
        x0, up = torch.from_numpy(inp["x0"]).cuda(), torch.from_numpy(inp["upstream"]).cuda()
        st.forward(x0)
        torch.cuda.synchronize()
        idxs.append([to_np(st.idx[l]).copy() for l in range(L)])
        batches.append((x0, up, inp))
    st.dW_gu.fill_(9.0); st.dW_down.fill_(9.0)              # the first micro-batch overwrites
    losses = st.accumulate_microbatches([(b[0], b[1]) for b in batches])
    torch.cuda.synchronize()
    prev = np.full(M, 1.0 / M)
    tot_pool = O.zeros_like_pool(pool)
    tot_wr = [0.0] * L
    for i, (_, _, inp) in enumerate(batches):
        res = O.stack_objective_and_grads(f64(inp["x0"]), routers, pool, k, st.c, synth.EPS, synth.ALPHA,
                                          f64(inp["upstream"]), forced_idx=idxs[i], fbar_prev=prev)
        assert abs(float(losses[i][0]) - res["loss_aux"]) <= 1e-5 * abs(res["loss_aux"])
        for n in tot_pool:
            tot_pool[n] += res["pool_grad"][n]
        for l in range(L):
            tot_wr[l] = tot_wr[l] + res["router_grads"][l]["dW_r"]
        prev = O.pool_aux_loss(res["counts"], res["S"], T, k, synth.ALPHA)[1]       # this batch's f-bar
    f = cfg["f"]
    assert rel_max(to_np(st.dW_gu)[:, :f], tot_pool["W_gate"]) < 1e-5
    assert rel_max(to_np(st.dW_gu)[:, f:], tot_pool["W_up"]) < 1e-5
    assert rel_max(to_np(st.dW_down), tot_pool["W_down"]) < 1e-5
    for l in range(L):
        assert rel_max(to_np(st.dW_r[l]), tot_wr[l]) < 1e-5
    assert rel_max(to_np(st.fbar_lag[0]), prev) < 1e-6
    st.ctx.check_status()
    st.close()


def test_recomputed_activations_give_the_same_step():
    """MoE-layer activation recompute: keeping only x_l and the routing state and rebuilding the
    permuted activations in backward reproduces the step bit for bit."""
    import torch
    cfg = small_cfg(dtype="bf16", d=256, f=384, M=16, k=2, L=3)
    T = 900
    inputs = synth.make_inputs(cfg, seed=12, T=T)
    x0 = torch.from_numpy(inputs["x0"]).cuda().bfloat16()
    up = torch.from_numpy(inputs["upstream"]).cuda().bfloat16()
    outs = []
    for recompute in (False, True):
        from paper_2605_06665_b200.stack import UniPoolStack
        st = UniPoolStack(cfg["L"], cfg["d"], cfg["f"], cfg["M"], cfg["k"], T, "bf16", 0, c=2.5, eps=synth.EPS,
                          alpha=synth.ALPHA, recompute=recompute)
        st.load(inputs["pool"], inputs["routers"])
        assert st.Xp.shape[0] == (1 if recompute else cfg["L"])
        st.zero_grad()
        dx0 = st.step(x0, up).clone()
        torch.cuda.synchronize()
        st.ctx.check_status()
        outs.append([t.clone() for t in (st.x[cfg["L"]], dx0, st.dW_gu, st.dW_down, st.dW_r)])
        st.close()
    for a, b in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a, b)
    assert rel_max(to_np(outs[1][4]), to_np(outs[0][4])) < 1e-5     # router dW: split-K add-reduce, order may differ
    assert outs[0][2].abs().max() > 0


@pytest.mark.parametrize("dtype,deferred", [("fp32", False), ("fp32", True), ("bf16", True)])
def test_sharing_scope_groups(dtype, deferred):
    """G = 2 sharing groups over L = 4 layers (the ablation's intermediate sharing scope): layers
    {0,1} share pool experts 0..7, layers {2,3} experts 8..15, each group with its own Eq. 5 loss.
    Whole step against the float64 oracle (forced to the GPU's routing)."""
    import torch
    cfg = small_cfg(dtype=dtype, d=128, f=192, M=16, k=2, L=4, groups=2)
    T = 400
    inputs = synth.make_inputs(cfg, seed=14, T=T)
    st = build_stack(cfg, inputs, T=T, deferred_wgrad=deferred)
    assert st.m == 8 and st.G == 2 and st.deferred_wgrad == deferred
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    x0 = torch.from_numpy(inputs["x0"]).cuda().to(tdt)
    up = torch.from_numpy(inputs["upstream"]).cuda().to(tdt)
    st.dW_gu.fill_(4.0); st.dW_down.fill_(4.0)
    st.step(x0, up, accumulate=False)
    torch.cuda.synchronize()
    st.ctx.check_status()
    pool, routers = oracle_params(inputs, 4)
    views = [synth.expert_base(cfg, l) for l in range(4)]
    assert views == [0, 0, 8, 8]
    idx = [to_np(st.idx[l]) for l in range(4)]
    if dtype == "fp32":
        res = O.stack_objective_and_grads(f64(inputs["x0"]), routers, pool, 2, st.c, synth.EPS, synth.ALPHA,
                                          f64(inputs["upstream"]), views, forced_idx=idx, aux_groups=[[0, 1], [2, 3]])
        tol = 1e-5
        assert rel_max(to_np(st.x[4]), res["caches"][-1]["x_next"]) < tol
        assert abs(float(st.loss.sum()) - res["loss_aux"]) <= 1e-5 * abs(res["loss_aux"])
        f = cfg["f"]
        assert rel_max(to_np(st.dW_gu)[:, :f], res["pool_grad"]["W_gate"]) < tol
        assert rel_max(to_np(st.dW_down), res["pool_grad"]["W_down"]) < tol
        for l in range(4):
            assert rel_max(to_np(st.dW_r[l]), res["router_grads"][l]["dW_r"]) < tol
    else:
        # bf16: the grouped one-pass weight gradient must equal the per-layer accumulation
        ref = build_stack(cfg, inputs, T=T, deferred_wgrad=False)
        ref.zero_grad()
        ref.step(x0, up)
        torch.cuda.synchronize()
        assert rel_max(to_np(st.dW_gu), to_np(ref.dW_gu)) < 1e-5
        assert rel_max(to_np(st.dW_down), to_np(ref.dW_down)) < 1e-5
        assert torch.equal(st.x[4], ref.x[4])
        ref.close()
    st.close()


@pytest.mark.parametrize("kw", [dict(M=8, k=2, L=4), dict(M=12, k=2, private=4, L=3), dict(M=40, k=8, d=64, f=64, L=2)])
def test_unique_experts_per_token(kw):
    """App. E's U(x) over the routing decisions of a real forward pass, bit-exact against the oracle."""
    import torch
    cfg = small_cfg(**kw)
    T, L = 257, cfg["L"]
    inputs = synth.make_inputs(cfg, seed=2, T=T)
    st = build_stack(cfg, inputs, T=T)
    st.forward(torch.from_numpy(inputs["x0"]).cuda())
    views = [synth.expert_base(cfg, l) for l in range(L)]
    base = torch.tensor(views, dtype=torch.int32, device="cuda") if cfg["private"] else None
    unique = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    total = torch.full((1,), 77, dtype=torch.int64, device="cuda")
    st.ctx.unique_experts(st.idx, base, L, T, unique, total)
    torch.cuda.synchronize()
    ref = O.unique_experts([to_np(st.idx[l]) for l in range(L)], views if cfg["private"] else None)
    assert (to_np(unique) == ref).all()
    assert int(total[0]) == int(ref.sum())
    if cfg["private"]:
        assert (ref == L * cfg["k"]).all()
    st.close()


def test_calibrate_c_on_device():
    from oracle import norm_router_c
    cfg = small_cfg()
    st = build_stack(cfg, synth.make_inputs(cfg, seed=0))
    for (E, k) in [(96, 2), (16, 2), (384, 8)]:
        got = st.ctx.calibrate_c(E, k, 200_000, seed=1)
        ref = norm_router_c.estimate_c(E, k, 200_000, seed=2)
        assert got >= 1.0 and abs(got - ref) / ref < 5e-3
    st.close()


def test_corrupt_routing_table_is_reported_not_faulted():
    """An out-of-range expert id is caught by the dispatch kernel's own bounds check:
    the assignment is dropped and the status word reports it."""
    import torch
    from paper_2605_06665_b200 import binding as B
    cfg = small_cfg()
    st = build_stack(cfg, synth.make_inputs(cfg, seed=0))
    st.forward_layer(0)
    st.idx[0, 5, 1] = 1000
    st.ctx.dispatch(st.x[0], cfg["T"], st.idx[0], cfg["M"], st.offsets[0], st.row_of[0], st.token_of[0],
                    st.tile_expert[0], st.Xp[0])
    with pytest.raises(B.UniPoolError) as ei:
        st.ctx.check_status()
    assert ei.value.code == -6
    assert int(st.row_of[0, 5, 1]) == -1
    st.ctx.check_status()          # cleared
    st.close()


def test_an_expired_device_wait_is_reported_and_the_context_stays_usable():
    """Every barrier wait in the GEMM and router pipelines is bounded.  The self-test launches one
    thread that waits a few microseconds on a barrier nobody arrives on: the wait gives up, the kernel
    returns normally, the status word reports the time-out once, and later calls work as before."""
    import torch
    from paper_2605_06665_b200 import binding as B
    cfg = small_cfg(dtype="bf16", d=128, f=128, M=8, k=2)
    inputs = synth.make_inputs(cfg, seed=1)
    st = build_stack(cfg, inputs)
    st.x[0].copy_(torch.from_numpy(inputs["x0"]))
    st.forward_layer(0)
    torch.cuda.synchronize()
    before = st.x[1].clone()
    st.ctx.check_status()
    st.ctx.selftest_wait(20_000)                     # about ten microseconds of SM clock
    torch.cuda.synchronize()                         # the kernel has returned: nothing is left waiting
    with pytest.raises(B.UniPoolError) as ei:
        st.ctx.check_status()
    assert ei.value.code == -5 and "site 99" in str(ei.value)
    st.ctx.check_status()                            # reported once, then cleared
    st.forward_layer(0)                              # the context still works, and gives the same result
    torch.cuda.synchronize()
    st.ctx.check_status()
    assert torch.equal(st.x[1], before)
    with pytest.raises(B.UniPoolError):
        st.ctx.selftest_wait(-1)                     # refused on the host
    st.close()



_GUARD_CHILD = r"""
import numpy as np, torch
from paper_2605_06665_b200 import binding as B, synth
from paper_2605_06665_b200.stack import UniPoolStack
cfg = dict(synth.CONFIGS["tiny_fp32"]); cfg.update(dtype="bf16", d=128, f=128, M=8, k=2, L=2, T=300)
inp = synth.make_inputs(cfg, seed=5)
st = UniPoolStack(cfg["L"], cfg["d"], cfg["f"], cfg["M"], cfg["k"], cfg["T"], "bf16", 0, c=2.0, device="cuda:0")
st.load(inp["pool"], inp["routers"])
x0 = torch.from_numpy(inp["x0"]).to("cuda:0", torch.bfloat16)
y = st.forward(x0)
st.aux_loss()
st.backward(torch.ones_like(y))
st.ctx.check_status()                       # a whole step leaves every band as it was filled
print("intact")
ws = st.ctx.workspace
assert int(ws[256]) == 0xA5                 # the first band follows the 256-byte status region
ws[300] = 0                                 # what a kernel writing past its region would do
try:
    st.ctx.check_status()
    print("missed")
except B.UniPoolError as e:
    print("caught", e.code, str(e))
st.ctx.check_status()                       # reported once, the word is cleared; the band stays altered
"""


@pytest.mark.gpu
def test_debug_guard_bands_survive_a_step_and_report_an_overwrite():
    """Debug aid (no paper counterpart): with UNIPOOL_DEBUG=1 the workspace regions are fenced by
    guard bands that unipool_check_status compares with their fill."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, UNIPOOL_DEBUG="1")
    out = subprocess.run([sys.executable, "-c", _GUARD_CHILD], cwd=root, env=env, capture_output=True, text=True)
    assert out.returncode != 0 or "intact" in out.stdout, out.stderr[-2000:]
    lines = out.stdout.strip().splitlines()
    assert lines[0] == "intact", out.stdout + out.stderr[-2000:]
    assert lines[1].startswith("caught -6") and "guard band behind workspace region 0" in lines[1], out.stdout
