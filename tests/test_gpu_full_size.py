"""GPU parity at the full workload sizes, in the launch configuration the benchmark times
(bf16, weight gradients of all layers contracted in one pass that overwrites the pool-gradient
buffers), against the CPU oracle on what the oracle can afford:

  * routing of EVERY token of every layer (logits, top-k under the margin rule, gates, counts,
    score sums) and the permutation maps, bit-exact;
  * the layer output x_{l+1} and the input gradient dx_l on a seeded sample of tokens per layer;
  * the pool weight gradient, accumulated over ALL layers, of a sample of experts that always
    holds the largest group, the smallest non-empty group and (if any) an expert that received no
    token anywhere (whose gradient must be exactly zero);
  * the balance loss.

Each layer's oracle consumes the GPU's own x_l and dx_{l+1} (converted to float64), so only that
layer's arithmetic is compared: bf16 rounding of x_l legitimately re-routes a few tokens per layer.
Tolerances as in the small-shape tests: 1e-2 of the largest reference magnitude for bf16 storage,
1e-5 for the fp32 quantities of the router and the balance loss.

The router, the maps and the balance loss are always evaluated in float64.  The expert path of the
978M-shaped workloads is evaluated by the oracle in float32 (its arithmetic follows the dtype of its
inputs): the sampled tokens of a layer touch every one of the 192 experts, and widening 14.5 GB of
weights to float64 once per layer and pass would take the oracle minutes per layer.  The operands
are bf16 values, so every product is exact in float32 and only the summation differs (relative
1e-6 or so against a bound of 1e-2).
"""
import numpy as np
import pytest

from oracle import unipool_oracle as O
from paper_2605_06665_b200 import synth
from parity_utils import build_stack, check_routing, f64, rel_max, to_np

pytestmark = pytest.mark.gpu

TOL = 1e-2
N_TOKENS = 1024         # sampled tokens per layer
N_EXPERTS = 3           # random experts on top of the three structural picks


def sampled_experts(total_counts, rng):
    """Router-local expert ids: largest group, smallest non-empty group, an empty one, a few random."""
    picks = [int(np.argmax(total_counts))]
    nz = np.nonzero(total_counts)[0]
    picks.append(int(nz[np.argmin(total_counts[nz])]))
    empty = np.nonzero(total_counts == 0)[0]
    if empty.size:
        picks.append(int(empty[0]))
    picks += [int(e) for e in rng.choice(len(total_counts), size=N_EXPERTS, replace=False)]
    return sorted(set(picks))


@pytest.mark.parametrize("name,L", [
    ("182m", None), ("182m_vanilla", None), ("182m_pool40", None), ("fine_zipf", None),
    ("182m_vanilla_softmax", None),
    ("978m", None), ("978m_pool128", None), ("978m_vanilla", None),
])
def test_full_size_sampled_parity(name, L):
    import torch
    cfg = dict(synth.CONFIGS[name])
    L = cfg["L"] if L is None else L
    T, k, d, f, M = cfg["T"], cfg["k"], cfg["d"], cfg["f"], cfg["M"]
    m = synth.router_width(cfg)
    mode = cfg.get("router", "norm")
    inputs = synth.make_inputs(cfg, seed=0, L=L)
    st = build_stack(cfg, inputs, L=L, deferred_wgrad=True)
    pool = inputs["pool"]                                   # float32 holding bf16 values
    ex = f64 if d <= 768 else (lambda a: np.asarray(a, dtype=np.float32))   # dtype of the oracle's expert path
    routers = [dict(W_r=f64(r["W_r"]), sigma=float(r["sigma"]),
                    bias=None if r["bias"] is None else f64(r["bias"])) for r in inputs["routers"]]
    c, eps, alpha = st.c, synth.EPS, synth.ALPHA
    rng = np.random.default_rng(123)
    st.x[0].copy_(torch.from_numpy(inputs["x0"]))

    # ---------------------------------------------------------------- forward, layer by layer
    routes, xs = [], []
    for l in range(L):
        st.forward_layer(l)
        torch.cuda.synchronize()
        x_l = f64(to_np(st.x[l]))
        xs.append(x_l)
        ref = O.route(x_l, routers[l]["W_r"], routers[l]["sigma"], c, eps, k, routers[l]["bias"], mode=mode)
        idx_gpu = to_np(st.idx[l])
        check_routing(idx_gpu, ref["z"], ref["idx"], k, mode)
        assert rel_max(to_np(st.z[l]), ref["z"]) < 1e-5
        ref = O.route(x_l, routers[l]["W_r"], routers[l]["sigma"], c, eps, k, routers[l]["bias"], forced_idx=idx_gpu,
                      mode=mode)
        assert rel_max(to_np(st.gate[l]), ref["g"]) < 1e-5
        assert (to_np(st.counts[l]) == ref["counts"]).all() and ref["counts"].sum() == T * k
        assert rel_max(to_np(st.score_sum[l]), ref["S"]) < 1e-5
        off, row_of, token_of = O.dispatch_map(idx_gpu, m, 128)
        assert (to_np(st.offsets[l]) == off).all()
        assert (to_np(st.row_of[l]) == row_of).all()
        used = int(off[-1])
        tok_gpu = to_np(st.token_of[l])
        assert (tok_gpu[:used] == token_of).all() and (tok_gpu[used:] == -1).all()
        tokens = np.sort(rng.choice(T, size=N_TOKENS, replace=False))
        y_ref = O.moe_layer_output(ex(x_l), idx_gpu, ex(ref["g"]), pool, synth.expert_base(cfg, l), tokens=tokens)
        got = f64(to_np(st.x[l + 1][torch.from_numpy(tokens).cuda()]))
        assert rel_max(got, x_l[tokens] + f64(y_ref)) < TOL
        # ... and at the scale of the expert outputs themselves (the residual stream can dwarf them): the
        # gate-weighted sum of the GPU's un-combined expert rows of the sampled tokens
        rows = torch.from_numpy(to_np(st.row_of[l])[tokens].astype(np.int64)).cuda()          # [n, k]
        y_rows = f64(to_np(st.Yp[st.slot(l)][rows.reshape(-1)])).reshape(len(tokens), k, d)
        assert rel_max(np.einsum("tj,tjd->td", f64(ref["g"])[tokens], y_rows), f64(y_ref)) < TOL
        ref["tokens"] = tokens
        routes.append(ref)

    # ---------------------------------------------------------------- balance loss
    st.aux_loss()
    torch.cuda.synchronize()
    counts = np.stack([r["counts"] for r in routes])
    S = np.stack([f64(to_np(st.score_sum[l])) for l in range(L)])
    if cfg["private"]:
        coefs = []
        for l in range(L):
            lo, _, co = O.pool_aux_loss(counts[l:l + 1], S[l:l + 1], T, k, alpha)
            assert abs(float(st.loss[l]) - lo) <= 1e-5 * abs(lo)
            coefs.append(co)
    else:
        lo, fb, co = O.pool_aux_loss(counts, S, T, k, alpha)
        assert abs(float(st.loss[0]) - lo) <= 1e-5 * abs(lo)
        assert rel_max(to_np(st.coef[0]), co) < 1e-5 and rel_max(to_np(st.fbar[0]), fb) < 1e-5
        coefs = [co] * L

    # ---------------------------------------------------------------- backward as the benchmark issues it
    if cfg["private"]:
        experts = {l: sampled_experts(counts[l], rng)[:3] for l in range(0, L, max(1, L // 3))}
    else:
        shared = sampled_experts(counts.sum(axis=0), rng)      # the same pool experts in every layer
        experts = {l: shared for l in range(L)}
    grad = {n: {} for n in ("W_gate", "W_up", "W_down")}
    for l, es in experts.items():
        for e in es:
            pe = synth.expert_base(cfg, l) + e
            for n in grad:
                grad[n].setdefault(pe, np.zeros(pool[n].shape[1:], dtype=ex(0.0).dtype))
    st.dW_gu.fill_(3.0); st.dW_down.fill_(-5.0)               # the overwriting pass must replace these
    st.zero_router_grad()
    dx_cur = torch.from_numpy(inputs["upstream"]).to(st.device, st.tdtype)
    for l in reversed(range(L)):
        dx_out = torch.empty_like(dx_cur)
        st.backward_layer(l, dx_cur, dx_out, overwrite=bool(cfg["private"]))
        torch.cuda.synchronize()
        r = routes[l]
        base = synth.expert_base(cfg, l)
        dxn = f64(to_np(dx_cur))
        tokens = r["tokens"]
        dx_e, dg = O.expert_path_backward(ex(xs[l]), r["idx"], ex(r["g"]), pool, ex(dxn), base, tokens=tokens)
        dx_e, dg = f64(dx_e), f64(dg)
        assert rel_max(to_np(st.dgate)[tokens], dg) < TOL
        rb = O.route_backward(xs[l][tokens], routers[l]["W_r"], routers[l]["sigma"], c, eps, r["z"][tokens],
                              r["n"][tokens], r["idx"][tokens], dg, coefs[l], mode=mode)
        got = f64(to_np(dx_out[torch.from_numpy(tokens).cuda()]))
        assert rel_max(got, dxn[tokens] + dx_e + rb["dx"]) < TOL
        if l in experts:
            O.expert_path_backward(ex(xs[l]), r["idx"], ex(r["g"]), pool, ex(dxn), base, grad, experts=experts[l])
        dx_cur = dx_out
    if st.deferred_wgrad:
        from paper_2605_06665_b200 import binding as B
        st.ctx.pool_wgrad(L, st.cap, st.offsets, st.Xp, st.A, st.dYp, st.dGU, 0, m, st.dW_gu, st.dW_down,
                          B.WGRAD_OVERWRITE)
    torch.cuda.synchronize()
    st.ctx.check_status()
    scale = {n: max(np.abs(g).max() for g in grad[n].values()) for n in grad}
    assert min(scale.values()) > 0
    for pe in grad["W_down"]:
        gu = f64(to_np(st.dW_gu[pe]))
        gd = f64(to_np(st.dW_down[pe]))
        assert np.abs(gu[:f] - grad["W_gate"][pe]).max() < TOL * scale["W_gate"], pe
        assert np.abs(gu[f:] - grad["W_up"][pe]).max() < TOL * scale["W_up"], pe
        assert np.abs(gd - grad["W_down"][pe]).max() < TOL * scale["W_down"], pe
        if not grad["W_down"][pe].any():
            assert not gu.any() and not gd.any(), "an expert without tokens must have a zero gradient"
    if not cfg["private"]:
        untouched = np.nonzero(counts.sum(axis=0) == 0)[0]
        for e in untouched[:8]:
            assert not to_np(st.dW_gu[int(e)]).any() and not to_np(st.dW_down[int(e)]).any()
    st.close()
    del st, dx_cur, dx_out
    torch.cuda.empty_cache()                                 # the next workload needs the memory
