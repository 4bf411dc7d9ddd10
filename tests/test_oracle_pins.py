"""Pins for the CPU oracle: hand-worked examples, brute force, closed forms,
invariants and finite differences.  None of these tests needs a GPU."""
import json
import math
import os

import numpy as np
import pytest

from oracle import brute, norm_router_c
from oracle import unipool_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")


def tiny_problem(seed=0, L=3, M=6, d=8, f=5, k=2, T=12, private=0, std=0.5, bias=False, mode="norm"):
    rng = np.random.default_rng(seed)
    m = private if private else M
    pool = dict(W_gate=rng.normal(0, std, (M, f, d)), W_up=rng.normal(0, std, (M, f, d)),
                W_down=rng.normal(0, std, (M, d, f)))
    routers = [dict(W_r=rng.normal(0, std, (m, d)), sigma=1.0 + 0.1 * l,
                    bias=(rng.normal(0, 0.3, m) if bias else None), mode=mode) for l in range(L)]
    x0 = rng.normal(0, 1, (T, d))
    up = rng.normal(0, 1, (T, d))
    views = [private * l for l in range(L)] if private else None
    return pool, routers, x0, up, views


# ---------------------------------------------------------------- hand examples
def test_golden_hand_examples():
    g = json.load(open(GOLDEN))
    ex = g["norm_router"]
    s, n = O.norm_router_scores(np.array([ex["z"]]), ex["sigma"], ex["c"], ex["eps"])
    np.testing.assert_allclose(s[0], ex["s"], rtol=0, atol=1e-15)
    assert n[0] == ex["n"]

    ex = g["pool_aux"]
    loss, fbar, coef = O.pool_aux_loss(np.array(ex["counts"]), np.array(ex["S"]), ex["T"], ex["k"], ex["alpha"])
    assert loss == pytest.approx(ex["loss"], rel=1e-14)
    np.testing.assert_allclose(fbar, ex["fbar"], rtol=1e-15)
    np.testing.assert_allclose(coef, ex["coef"], rtol=1e-15)

    ex = g["switch_aux"]
    assert O.switch_aux_loss(np.array(ex["counts"]), np.array(ex["S"]), ex["T"], ex["k"], ex["alpha"]) == \
        pytest.approx(ex["loss"], rel=1e-14)

    ex = g["swiglu"]
    _, _, _, Y = O.expert_ffn(np.array([ex["h"]]), np.array(ex["W_gate"]), np.array(ex["W_up"]),
                              np.array(ex["W_down"]))
    np.testing.assert_allclose(Y[0], ex["y"], rtol=1e-15)
    yb = brute.swiglu_expert_token(ex["h"], ex["W_gate"], ex["W_up"], ex["W_down"])
    np.testing.assert_allclose(yb, ex["y"], rtol=1e-15)


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("private,bias", [(0, False), (0, True), (2, False)])
def test_vectorised_forward_matches_per_token_loops(private, bias):
    pool, routers, x0, _, views = tiny_problem(seed=1, private=private, bias=bias)
    k, c, eps = 2, 1.7, 1e-6
    caches = O.stack_forward(x0, routers, pool, k, c, eps, views)
    to_list = lambda a: a.tolist()
    b = brute.stack_forward(to_list(x0), [dict(W_r=to_list(r["W_r"]), sigma=r["sigma"],
                                               bias=None if r["bias"] is None else to_list(r["bias"]))
                                          for r in routers],
                            {n: to_list(w) for n, w in pool.items()}, k, c, eps, views)
    for cache, bl in zip(caches, b):
        assert cache["idx"].tolist() == bl["idx"]
        np.testing.assert_allclose(cache["g"], bl["g"], rtol=1e-12, atol=1e-14)
        assert cache["counts"].tolist() == bl["counts"]
        np.testing.assert_allclose(cache["S"], bl["S"], rtol=1e-12)
        np.testing.assert_allclose(cache["x_next"], bl["x_next"], rtol=1e-10, atol=1e-12)
    counts = np.stack([cc["counts"] for cc in caches])
    S = np.stack([cc["S"] for cc in caches])
    if not private:
        loss, _, _ = O.pool_aux_loss(counts, S, x0.shape[0], k, 0.01)
        assert loss == pytest.approx(brute.pool_aux_loss(counts.tolist(), S.tolist(), x0.shape[0], k, 0.01),
                                     rel=1e-12)


# ---------------------------------------------------------------- NormRouter
def test_norm_router_invariants():
    rng = np.random.default_rng(3)
    z = rng.normal(0, 2.0, (2000, 64))
    sigma, c = 1.3, 2.1
    s, n = O.norm_router_scores(z, sigma, c, 0.0)
    assert (s >= 0).all()
    assert (np.sum((s / (sigma * c)) ** 2, axis=1) <= 1 + 1e-12).all()
    # bounded regardless of input scale: invariant under z -> lambda z (eps = 0)
    s2, _ = O.norm_router_scores(37.5 * z, sigma, c, 0.0)
    np.testing.assert_allclose(s2, s, rtol=1e-12, atol=1e-15)
    # about half of the experts get a zero score on symmetric logits
    assert abs((s == 0).mean() - 0.5) < 0.01
    # the norm runs over the whole logit vector, negatives included
    np.testing.assert_allclose(n, np.linalg.norm(z, axis=1), rtol=1e-14)
    # M = 1: s = sigma c 1{z>0} |z| / (|z| + eps)
    z1 = np.array([[2.0], [-3.0], [0.0]])
    s1, _ = O.norm_router_scores(z1, sigma, c, 0.5)
    np.testing.assert_allclose(s1[:, 0], [sigma * c * 2.0 / 2.5, 0.0, 0.0], rtol=1e-15)


def test_top_k_against_full_sort_and_ties():
    rng = np.random.default_rng(4)
    s = rng.random((300, 17))
    idx = O.top_k(s, 4)
    for t in range(s.shape[0]):
        ref = sorted(range(17), key=lambda i: (-s[t, i], i))[:4]
        assert idx[t].tolist() == ref
    # equal scores: lowest index wins, in index order
    tie = np.array([[0.5, 0.9, 0.5, 0.9, 0.1], [0.0, 0.0, 0.0, 0.0, 0.0]])
    assert O.top_k(tie, 3).tolist() == [[1, 3, 0], [0, 1, 2]]
    # all logits negative -> all scores zero -> experts 0..k-1
    z = -np.abs(rng.normal(0, 1, (5, 8))) - 0.1
    r = O.route(rng.normal(0, 1, (5, 3)), np.zeros((8, 3)), 1.0, 1.0, 1e-6, 3, bias=z[0])
    assert (r["idx"] == np.array([0, 1, 2])).all() and (r["g"] == 0).all()


def test_route_counts_and_gates():
    rng = np.random.default_rng(5)
    T, d, M, k = 257, 16, 24, 3
    r = O.route(rng.normal(0, 1, (T, d)), rng.normal(0, 0.3, (M, d)), 0.9, 2.5, 1e-6, k)
    assert r["counts"].sum() == T * k
    assert all(len(set(row)) == k for row in r["idx"].tolist())
    assert (np.diff(r["g"], axis=1) <= 0).all()            # descending scores
    for t in range(T):
        for j in range(k):
            assert r["g"][t, j] == r["s"][t, r["idx"][t, j]]
    np.testing.assert_allclose(r["S"], r["s"].sum(0))
    # gates are not renormalised: bounded by sigma*c in L2, not summing to one
    assert (np.sum((r["g"] / (0.9 * 2.5)) ** 2, axis=1) <= 1 + 1e-12).all()


# ---------------------------------------------------------------- calibration constant
def test_calibration_constant_c():
    # all-positive vector with k = E: ReLU changes nothing, the unit vector has norm 1
    x = np.abs(np.random.default_rng(0).normal(0, 1, (50, 8))) + 0.01
    np.testing.assert_allclose(norm_router_c.topk_norm(x, 8), 1.0, rtol=1e-14)
    # E = 2, k = 1, x = (3, 4): y = (.6, .8), top-1 norm .8
    np.testing.assert_allclose(norm_router_c.topk_norm(np.array([[3.0, 4.0]]), 1), 0.8, rtol=1e-15)
    c_a = norm_router_c.estimate_c(96, 2, 100_000, seed=0)
    c_b = norm_router_c.estimate_c(96, 2, 100_000, seed=1)
    assert c_a >= 1.0 and abs(c_a - c_b) / c_a < 3e-3
    # c makes the selected scores of an untrained router approximately unit length
    rng = np.random.default_rng(9)
    r = O.route(rng.normal(0, 1, (4000, 64)), rng.normal(0, 0.02, (96, 64)), 1.0, c_a, 1e-6, 2)
    mean_norm = np.sqrt((r["g"] ** 2).sum(1)).mean()
    assert abs(mean_norm - 1.0) < 0.05


# ---------------------------------------------------------------- dense special case
def test_single_expert_reduces_to_dense_swiglu():
    rng = np.random.default_rng(6)
    T, d, f = 9, 7, 11
    x = rng.normal(0, 1, (T, d))
    pool = dict(W_gate=rng.normal(0, 0.5, (1, f, d)), W_up=rng.normal(0, 0.5, (1, f, d)),
                W_down=rng.normal(0, 0.5, (1, d, f)))
    y = O.moe_layer_output(x, np.zeros((T, 1), np.int32), np.ones((T, 1)), pool)
    ref = np.zeros((T, d))
    for t in range(T):                              # textbook triple loop
        a = np.zeros(f)
        for p in range(f):
            gg = sum(pool["W_gate"][0][p, q] * x[t, q] for q in range(d))
            uu = sum(pool["W_up"][0][p, q] * x[t, q] for q in range(d))
            a[p] = gg / (1 + math.exp(-gg)) * uu
        for q in range(d):
            ref[t, q] = sum(pool["W_down"][0][q, p] * a[p] for p in range(f))
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- permutation
@pytest.mark.parametrize("align", [1, 4, 128])
def test_dispatch_map_is_a_stable_grouping(align):
    rng = np.random.default_rng(7)
    T, k, M = 301, 3, 13
    idx = np.stack([rng.permutation(M)[:k] for _ in range(T)]).astype(np.int32)
    idx[idx == 5] = 6                                # expert 5 empty (duplicates in a row are fine here)
    offsets, row_of, token_of = O.dispatch_map(idx, M, align)
    counts = np.bincount(idx.reshape(-1), minlength=M)
    assert (offsets % align == 0).all() and offsets[0] == 0
    assert (np.diff(offsets) == (counts + align - 1) // align * align).all()
    assert len(set(row_of.reshape(-1).tolist())) == T * k          # injective
    flat = [(int(idx[t, j]), t, j) for t in range(T) for j in range(k)]
    for e in range(M):
        rows = [int(row_of[t, j]) for (ee, t, j) in flat if ee == e]
        assert rows == list(range(int(offsets[e]), int(offsets[e]) + counts[e]))   # stable, contiguous
        assert (token_of[offsets[e] + counts[e]:offsets[e + 1]] == -1).all()
    assert (token_of[row_of] == np.arange(T)[:, None]).all()
    # k = 1, unit gates, identity experts: combine(dispatch(x)) == x exactly
    x = rng.normal(0, 1, (T, 4))
    off1, row1, tok1 = O.dispatch_map(idx[:, :1], M, align)
    Xp = np.where(tok1[:, None] >= 0, x[np.maximum(tok1, 0)], 0.0)
    assert (Xp[row1[:, 0]] == x).all()


# ---------------------------------------------------------------- balance loss
def test_aux_loss_identities():
    rng = np.random.default_rng(8)
    L, M, T, k, alpha = 5, 12, 640, 2, 0.02
    counts = rng.multinomial(T * k, np.ones(M) / M, size=L)
    S = rng.random((L, M)) * T
    loss, fbar, coef = O.pool_aux_loss(counts, S, T, k, alpha)
    # Eq. 5 == Eq. 6 (App. G)
    assert loss == pytest.approx(O.pool_aux_loss_decomposed(counts, S, T, k, alpha), rel=1e-13)
    assert fbar.sum() == pytest.approx(1.0, rel=1e-13)
    # L = 1 is the per-layer loss of Eq. 3
    l1, _, _ = O.pool_aux_loss(counts[:1], S[:1], T, k, alpha)
    assert l1 == pytest.approx(O.switch_aux_loss(counts[0], S[0], T, k, alpha), rel=1e-13)
    # uniform utilisation: loss = alpha * sum_i Pbar_i
    cu = np.full((L, M), T * k // M)
    lu, _, _ = O.pool_aux_loss(cu, S, T * k // M * M // k, k, alpha)
    Tu = T * k // M * M // k
    assert lu == pytest.approx(alpha * (S / Tu).mean(0).sum(), rel=1e-13)
    # constant mean score p: loss = alpha * M * p (f sums to one)
    lp, _, _ = O.pool_aux_loss(counts, np.full((L, M), 0.3 * T), T, k, alpha)
    assert lp == pytest.approx(alpha * M * 0.3, rel=1e-13)
    # uniform utilisation and scores that sum to one: the closed-form minimum alpha
    lm, _, _ = O.pool_aux_loss(cu, np.full((L, M), Tu / M), Tu, k, alpha)
    assert lm == pytest.approx(alpha, rel=1e-13)
    # any non-uniform utilisation paired with matching scores is above the minimum
    p = rng.dirichlet(np.ones(M))
    cn = np.round(p * T * k).astype(int)
    Tn = cn.sum() / k
    ln, _, _ = O.pool_aux_loss(cn[None], (p * Tn)[None], Tn, k, alpha)
    assert ln > alpha
    # the gradient w.r.t. any score s^(l)_{t,i} is the constant alpha M fbar_i / (L T)
    dS = 1e-3
    for (l, i) in [(0, 0), (3, 7)]:
        S2 = S.copy()
        S2[l, i] += dS
        l2, _, _ = O.pool_aux_loss(counts, S2, T, k, alpha)
        assert (l2 - loss) / dS == pytest.approx(coef[i], rel=1e-8)
    np.testing.assert_allclose(coef, alpha * M * fbar / (L * T), rtol=1e-14)
    # one-step-behind: a supplied fbar replaces this batch's
    prev = rng.dirichlet(np.ones(M))
    lo, fb_now, co = O.pool_aux_loss(counts, S, T, k, alpha, fbar_prev=prev)
    assert lo == pytest.approx(alpha * M * np.sum(prev * (S / T).mean(0)), rel=1e-13)
    np.testing.assert_allclose(fb_now, fbar)
    # ... also in the gradient: with the lagged fbar held constant the loss is linear in the scores,
    # d loss / d s^(l)_{t,i} = alpha M prev_i / (L T)  (App. G: only P carries gradient)
    np.testing.assert_allclose(co, alpha * M * prev / (L * T), rtol=1e-14)
    for (l, i) in [(1, 2), (2, 5)]:
        S2 = S.copy()
        S2[l, i] += dS
        l2, _, _ = O.pool_aux_loss(counts, S2, T, k, alpha, fbar_prev=prev)
        assert (l2 - lo) / dS == pytest.approx(co[i], rel=1e-8)


# ---------------------------------------------------------------- softmax router (the paper's baseline router)
def test_softmax_router_hand_example():
    ex = json.load(open(GOLDEN))["softmax_router"]
    z = np.array([ex["z"]])
    s, lse = O.softmax_router_scores(z)
    np.testing.assert_allclose(s[0], ex["s"], rtol=1e-14)
    assert lse[0] == pytest.approx(ex["lse"], rel=1e-14)
    r = O.route(np.eye(3)[:1], np.zeros((3, 3)), 1.0, 1.0, 1e-6, 2, bias=z[0], mode="softmax")
    assert r["idx"][0].tolist() == ex["top2"]
    np.testing.assert_allclose(r["g"][0], ex["gates"], rtol=1e-14)


def test_softmax_router_against_library_and_closed_forms():
    from scipy.special import logsumexp, softmax
    rng = np.random.default_rng(5)
    z = rng.normal(0, 3, (40, 11))
    z[3] += 700.0                                      # would overflow exp() without the max subtraction
    s, lse = O.softmax_router_scores(z)
    np.testing.assert_allclose(s, softmax(z, axis=1), rtol=1e-13, atol=0)
    np.testing.assert_allclose(lse, logsumexp(z, axis=1), rtol=1e-13)
    np.testing.assert_allclose(s.sum(1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(O.softmax_router_scores(z - 17.5)[0], s, rtol=1e-12)       # shift invariance
    np.testing.assert_allclose(O.softmax_router_scores(np.full((2, 8), 0.3))[0], 1.0 / 8)  # equal logits
    # two experts: the logistic function of the logit difference
    z2 = rng.normal(0, 2, (9, 2))
    np.testing.assert_allclose(O.softmax_router_scores(z2)[0][:, 0], 1 / (1 + np.exp(z2[:, 1] - z2[:, 0])), rtol=1e-13)
    # exp is increasing: the softmax top-k is the top-k of the logits, gates are the probabilities
    x = rng.normal(0, 1, (30, 6))
    W = rng.normal(0, 1, (11, 6))
    b = rng.normal(0, 1, 11)
    r = O.route(x, W, 123.0, 456.0, 0.5, 3, bias=b, mode="softmax")   # sigma, c, eps play no part
    zz = x @ W.T + b
    np.testing.assert_array_equal(r["idx"], np.argsort(-zz, axis=1, kind="stable")[:, :3])
    np.testing.assert_allclose(r["g"], np.take_along_axis(softmax(zz, axis=1), r["idx"].astype(np.int64), 1), rtol=1e-13)
    np.testing.assert_allclose(r["S"].sum(), 30.0, rtol=1e-13)          # every token's probabilities sum to one
    assert r["counts"].sum() == 30 * 3
    # with probabilities, uniform routing reaches the Switch minimum of the balance loss: alpha
    counts = np.full((2, 8), 5)
    S = np.full((2, 8), 20 / 8.0)
    loss, _, _ = O.pool_aux_loss(counts, S, 20, 2, 0.01)
    assert loss == pytest.approx(0.01, rel=1e-13)


def test_softmax_backward_is_the_textbook_jacobian():
    rng = np.random.default_rng(6)
    T, M, d, k = 5, 7, 4, 2
    x = rng.normal(0, 1, (T, d))
    W = rng.normal(0, 1, (M, d))
    r = O.route(x, W, 1.0, 1.0, 1e-6, k, mode="softmax")
    dg = rng.normal(0, 1, (T, k))
    coef = rng.normal(0, 1, M)
    rb = O.route_backward(x, W, 1.0, 1.0, 1e-6, r["z"], r["n"], r["idx"], dg, coef, mode="softmax")
    for t in range(T):
        ds = coef.copy()
        for j in range(k):
            ds[r["idx"][t, j]] += dg[t, j]
        s = r["s"][t]
        jac = np.diag(s) - np.outer(s, s)               # d s_i / d z_m
        np.testing.assert_allclose(rb["dz"][t], jac.T @ ds, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(rb["dW_r"], sum(np.outer(rb["dz"][t], x[t]) for t in range(T)), rtol=1e-12)
    np.testing.assert_allclose(rb["dx"], np.stack([W.T @ rb["dz"][t] for t in range(T)]), rtol=1e-12)
    assert rb["dsigma"] == 0.0
    np.testing.assert_allclose(rb["dz"].sum(1), 0.0, atol=1e-14)          # probabilities sum to a constant


# ---------------------------------------------------------------- backward
def _objective(x0, routers, pool, k, c, eps, alpha, up, views, forced, fbar_prev, n_view):
    caches = O.stack_forward(x0, routers, pool, k, c, eps, views, forced)
    counts = np.stack([cc["counts"] for cc in caches])
    S = np.stack([cc["S"] for cc in caches])
    T = x0.shape[0]
    if views is None:
        aux, _, _ = O.pool_aux_loss(counts, S, T, k, alpha, fbar_prev)
    else:
        aux = sum(O.switch_aux_loss(counts[l], S[l], T, k, alpha) for l in range(len(routers)))
    return float(np.sum(up * caches[-1]["x_next"]) + aux), [cc["idx"] for cc in caches]


@pytest.mark.parametrize("private,bias,mode", [(0, False, "norm"), (0, True, "norm"), (2, False, "norm"),
                                               (0, True, "softmax"), (2, False, "softmax")])
def test_backward_matches_central_finite_differences(private, bias, mode):
    pool, routers, x0, up, views = tiny_problem(seed=11, L=3, M=6, d=8, f=5, k=2, T=10,
                                                private=private, bias=bias, mode=mode)
    k, c, eps, alpha = 2, 1.9, 1e-6, 0.5          # a large alpha makes the balance term visible
    res = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up, views, n_view=private)
    base_idx = [cc["idx"] for cc in res["caches"]]
    J0, _ = _objective(x0, routers, pool, k, c, eps, alpha, up, views, None, None, private)
    assert J0 == pytest.approx(res["J"], rel=1e-13)
    h = 1e-6
    rng = np.random.default_rng(0)

    def fd(arr, pos):
        old = arr[pos]
        arr[pos] = old + h
        Jp, ip = _objective(x0, routers, pool, k, c, eps, alpha, up, views, None, None, private)
        arr[pos] = old - h
        Jm, im = _objective(x0, routers, pool, k, c, eps, alpha, up, views, None, None, private)
        arr[pos] = old
        for a, b, c0 in zip(ip, im, base_idx):          # routing must not move inside the stencil
            assert (a == c0).all() and (b == c0).all()
        return (Jp - Jm) / (2 * h)

    checked = 0
    for name in ("W_gate", "W_up", "W_down"):
        used = np.unique(np.concatenate([(views[l] if views else 0) + cc["idx"].reshape(-1)
                                         for l, cc in enumerate(res["caches"])]))
        for e in used[:4]:
            pos = (int(e),) + tuple(int(rng.integers(0, s)) for s in pool[name].shape[1:])
            assert fd(pool[name], pos) == pytest.approx(res["pool_grad"][name][pos], rel=2e-5, abs=1e-8)
            checked += 1
    for l in range(len(routers)):
        W = routers[l]["W_r"]
        for _ in range(3):
            pos = tuple(int(rng.integers(0, s)) for s in W.shape)
            assert fd(W, pos) == pytest.approx(res["router_grads"][l]["dW_r"][pos], rel=2e-5, abs=1e-8)
        sig = np.array([routers[l]["sigma"]])
        routers[l]["sigma"] = sig                      # make it perturbable in place
        got = fd(sig, 0)
        routers[l]["sigma"] = float(sig[0])
        assert got == pytest.approx(res["router_grads"][l]["dsigma"], rel=2e-5, abs=1e-8)
    for _ in range(6):
        pos = tuple(int(rng.integers(0, s)) for s in x0.shape)
        assert fd(x0, pos) == pytest.approx(res["dx0"][pos], rel=2e-5, abs=1e-8)
    assert checked >= 9


def test_sharing_scope_groups_interpolate_between_pool_and_private():
    """G pools over depth: G = 1 is the shared pool (Eq. 5), G = L the layer-private layout
    (sum of Eq. 3), and for G = 2 the gradient of the grouped objective matches finite differences."""
    pool, routers, x0, up, _ = tiny_problem(seed=5, L=4, M=6, d=8, f=5, k=2, T=10)
    k, c, eps, alpha = 2, 1.9, 1e-6, 0.5
    one = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up)
    g1 = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up, views=[0] * 4,
                                     aux_groups=[[0, 1, 2, 3]])
    assert g1["J"] == pytest.approx(one["J"], rel=1e-14)
    np.testing.assert_allclose(g1["pool_grad"]["W_up"], one["pool_grad"]["W_up"], rtol=1e-12, atol=1e-14)
    # G = L with 4 private experts of 6... use a pool of 8 = 4 layers x 2 experts
    pool8, routers8, x0, up, views = tiny_problem(seed=6, L=4, M=8, d=8, f=5, k=2, T=10, private=2)
    priv = O.stack_objective_and_grads(x0, routers8, pool8, k, c, eps, alpha, up, views, n_view=2)
    gL = O.stack_objective_and_grads(x0, routers8, pool8, k, c, eps, alpha, up, views,
                                     aux_groups=[[0], [1], [2], [3]])
    assert gL["J"] == pytest.approx(priv["J"], rel=1e-14)
    np.testing.assert_allclose(gL["router_grads"][2]["dW_r"], priv["router_grads"][2]["dW_r"], rtol=1e-12)
    # G = 2: layers {0,1} share experts 0..3, layers {2,3} share experts 4..7; routers score 4 experts
    rng = np.random.default_rng(3)
    routers2 = [dict(W_r=rng.normal(0, 0.5, (4, 8)), sigma=1.0 + 0.1 * l, bias=None) for l in range(4)]
    views2, groups2 = [0, 0, 4, 4], [[0, 1], [2, 3]]
    res = O.stack_objective_and_grads(x0, routers2, pool8, k, c, eps, alpha, up, views2, aux_groups=groups2)
    base_idx = [cc["idx"] for cc in res["caches"]]

    def J():
        r = O.stack_objective_and_grads(x0, routers2, pool8, k, c, eps, alpha, up, views2, aux_groups=groups2)
        for a, b in zip(r["caches"], base_idx):
            assert (a["idx"] == b).all()
        return r["J"]

    def fd(arr, pos, h=1e-6):
        old = arr[pos]
        arr[pos] = old + h; jp = J()
        arr[pos] = old - h; jm = J()
        arr[pos] = old
        return (jp - jm) / (2 * h)

    used = np.unique(np.concatenate([views2[l] + cc["idx"].reshape(-1) for l, cc in enumerate(res["caches"])]))
    for e in used[:5]:
        pos = (int(e), int(rng.integers(0, 5)), int(rng.integers(0, 8)))
        assert fd(pool8["W_gate"], pos) == pytest.approx(res["pool_grad"]["W_gate"][pos], rel=2e-5, abs=1e-8)
    for l in range(4):
        pos = (int(rng.integers(0, 4)), int(rng.integers(0, 8)))
        assert fd(routers2[l]["W_r"], pos) == pytest.approx(res["router_grads"][l]["dW_r"][pos], rel=2e-5, abs=1e-8)


def test_data_parallel_replicas_sum_to_the_whole_batch():
    """Token shards with statistics summed over the replicas: the balance loss is the whole batch's
    and the replicas' gradients add up to the whole batch's gradient (routing is per token, the
    objective a sum over tokens plus a loss of batch statistics)."""
    pool, routers, x0, up, views = tiny_problem(seed=21, L=3, M=6, d=8, f=5, k=2, T=12, bias=True)
    k, c, eps, alpha = 2, 1.7, 1e-6, 0.3
    whole = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up)
    shards = [slice(0, 6), slice(6, 12)]
    local = [O.stack_objective_and_grads(x0[s], routers, pool, k, c, eps, alpha, up[s]) for s in shards]
    # the layer inputs of a shard are the whole batch's rows: statistics add up exactly
    counts = sum(r["counts"] for r in local)
    S = sum(r["S"] for r in local)
    assert (counts == whole["counts"]).all()
    np.testing.assert_allclose(S, whole["S"], rtol=1e-13)
    reps = [O.stack_objective_and_grads(x0[s], routers, pool, k, c, eps, alpha, up[s],
                                        replica_stats=lambda cn, ss: (counts, S, 12)) for s in shards]
    for r in reps:
        assert r["loss_aux"] == pytest.approx(whole["loss_aux"], rel=1e-13)
    # without the summed statistics the shards' losses do NOT average to the whole batch's
    assert abs(0.5 * (local[0]["loss_aux"] + local[1]["loss_aux"]) - whole["loss_aux"]) > 1e-6
    for name in ("W_gate", "W_up", "W_down"):
        np.testing.assert_allclose(reps[0]["pool_grad"][name] + reps[1]["pool_grad"][name],
                                   whole["pool_grad"][name], rtol=1e-10, atol=1e-13)
    for l in range(3):
        np.testing.assert_allclose(reps[0]["router_grads"][l]["dW_r"] + reps[1]["router_grads"][l]["dW_r"],
                                   whole["router_grads"][l]["dW_r"], rtol=1e-10, atol=1e-13)
        assert reps[0]["router_grads"][l]["dsigma"] + reps[1]["router_grads"][l]["dsigma"] == pytest.approx(
            whole["router_grads"][l]["dsigma"], rel=1e-10)
    np.testing.assert_allclose(np.concatenate([r["dx0"] for r in reps]), whole["dx0"], rtol=1e-10, atol=1e-13)


def test_data_parallel_replicas_with_one_step_behind_fbar():
    """With the lagged f-bar (App. G) a replica needs no statistic of the other replicas for the current
    micro-batch: its loss share (own score sums over the whole batch's token count) and its gradients
    add up, over the replicas, to the whole batch's."""
    pool, routers, x0, up, views = tiny_problem(seed=31, L=3, M=6, d=8, f=5, k=2, T=12)
    k, c, eps, alpha = 2, 1.7, 1e-6, 0.3
    fbar_prev = np.random.default_rng(1).dirichlet(np.ones(6))
    whole = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up, fbar_prev=fbar_prev)
    reps = [O.stack_objective_and_grads(x0[s], routers, pool, k, c, eps, alpha, up[s], fbar_prev=fbar_prev,
                                        replica_stats=lambda cn, S: (cn, S, 12)) for s in (slice(0, 6), slice(6, 12))]
    assert reps[0]["loss_aux"] + reps[1]["loss_aux"] == pytest.approx(whole["loss_aux"], rel=1e-13)
    for name in ("W_gate", "W_up", "W_down"):
        np.testing.assert_allclose(reps[0]["pool_grad"][name] + reps[1]["pool_grad"][name],
                                   whole["pool_grad"][name], rtol=1e-9, atol=1e-12)
    for l in range(3):
        np.testing.assert_allclose(reps[0]["router_grads"][l]["dW_r"] + reps[1]["router_grads"][l]["dW_r"],
                                   whole["router_grads"][l]["dW_r"], rtol=1e-9, atol=1e-12)
    # the next micro-batch's f-bar is the sum of the replicas' counts over the whole batch's assignments
    fb = sum(r["counts"].sum(0) for r in reps) / (3 * 12 * k)
    np.testing.assert_allclose(fb, whole["counts"].sum(0) / (3 * 12 * k))
    assert fb.sum() == pytest.approx(1.0)


def test_unique_expert_accounting():
    """App. E: private experts give U = L exactly for top-1 (L k for top-k); a shared pool gives
    1 <= U <= min(M, L k); a hand case; and U equals the row-wise count of a dense indicator matrix."""
    rng = np.random.default_rng(0)
    L, T, k, M = 5, 40, 1, 7
    idx = [rng.integers(0, 3, (T, k)).astype(np.int32) for _ in range(L)]
    assert (O.unique_experts(idx, views=[3 * l for l in range(L)]) == L).all()        # vanilla: exactly L
    U = O.unique_experts(idx)
    assert U.min() >= 1 and U.max() <= 3
    hand = [np.array([[0, 1]]), np.array([[1, 2]]), np.array([[0, 2]])]                   # top-2, 3 layers
    assert O.unique_experts(hand)[0] == 3
    assert O.unique_experts(hand, views=[0, 3, 6])[0] == 6
    idx2 = [np.stack([rng.permutation(M)[:2] for _ in range(T)]).astype(np.int32) for _ in range(L)]
    dense = np.zeros((T, M), bool)
    for a in idx2:
        for j in range(2):
            dense[np.arange(T), a[:, j]] = True
    assert (O.unique_experts(idx2) == dense.sum(axis=1)).all()


def test_shared_pool_gradient_is_the_sum_over_layers():
    """Each shared expert accumulates gradient from all L layers (Sec. 3): running the
    layers' backward passes one at a time into separate buffers and adding them gives
    the buffer that all layers accumulated into."""
    pool, routers, x0, up, _ = tiny_problem(seed=12, L=4, std=0.3)
    k, c, eps, alpha = 2, 1.9, 1e-6, 0.01
    res = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, up)
    total = O.zeros_like_pool(pool)
    for l in reversed(range(4)):
        g_l = O.zeros_like_pool(pool)
        cc = res["caches"][l]
        dx_next = up if l == 3 else res["router_grads"][l + 1]["dx"]
        O.expert_path_backward(cc["x"], cc["idx"], cc["g"], pool, dx_next, 0, g_l)
        for n in total:
            total[n] += g_l[n]
        # an expert no token of this layer reaches gets exactly zero from this layer
        unused = np.setdiff1d(np.arange(6), np.unique(cc["idx"]))
        for e in unused:
            assert not g_l["W_down"][e].any()
    for n in total:
        np.testing.assert_allclose(total[n], res["pool_grad"][n], rtol=1e-12, atol=1e-14)


def test_private_layout_equals_independent_layers():
    """Eq. 1: with views, layer l only touches its own experts, and its result is
    that of a stand-alone MoE layer holding just those experts."""
    pool, routers, x0, up, views = tiny_problem(seed=13, L=3, M=6, private=2)
    k, c, eps = 2, 1.5, 1e-6
    caches = O.stack_forward(x0, routers, pool, k, c, eps, views)
    for l, cc in enumerate(caches):
        own = {n: w[2 * l:2 * l + 2] for n, w in pool.items()}
        alone = O.layer_forward(cc["x"], routers[l], own, k, c, eps, 0)
        np.testing.assert_array_equal(alone["x_next"], cc["x_next"])
    res = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, 0.01, up, views, n_view=2)
    assert res["loss_aux"] == pytest.approx(
        sum(O.switch_aux_loss(cc["counts"], cc["S"], x0.shape[0], k, 0.01) for cc in caches), rel=1e-13)


def test_restricted_evaluation_matches_full():
    pool, routers, x0, up, _ = tiny_problem(seed=14, L=1, T=40)
    k, c, eps = 2, 1.5, 1e-6
    cc = O.layer_forward(x0, routers[0], pool, k, c, eps)
    tok = [3, 17, 5, 39]
    np.testing.assert_allclose(O.moe_layer_output(x0, cc["idx"], cc["g"], pool, tokens=tok), cc["y"][tok],
                               rtol=1e-13, atol=1e-15)
    full = O.zeros_like_pool(pool)
    dx, dg = O.expert_path_backward(x0, cc["idx"], cc["g"], pool, up, 0, full)
    dxs, dgs = O.expert_path_backward(x0, cc["idx"], cc["g"], pool, up, tokens=tok)
    np.testing.assert_allclose(dxs, dx[tok], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dgs, dg[tok], rtol=1e-13, atol=1e-15)
    part = O.zeros_like_pool(pool)
    O.expert_path_backward(x0, cc["idx"], cc["g"], pool, up, 0, part, experts=[1, 4])
    for n in part:
        np.testing.assert_allclose(part[n][[1, 4]], full[n][[1, 4]], rtol=1e-13, atol=1e-15)
        assert not part[n][[0, 2, 3, 5]].any()


def test_float32_mode_tracks_float64():
    pool, routers, x0, up, _ = tiny_problem(seed=15, L=2, T=64, std=0.2)
    k, c, eps = 2, 1.5, 1e-6
    r64 = O.stack_objective_and_grads(x0, routers, pool, k, c, eps, 0.01, up)
    f32 = lambda a: a.astype(np.float32)
    pool32 = {n: f32(w) for n, w in pool.items()}
    routers32 = [dict(W_r=f32(r["W_r"]), sigma=r["sigma"], bias=None) for r in routers]
    forced = [cc["idx"] for cc in r64["caches"]]
    r32 = O.stack_objective_and_grads(f32(x0), routers32, pool32, k, c, eps, 0.01, f32(up), forced_idx=forced)
    assert r32["dx0"].dtype == np.float32
    for n in pool:
        ref = r64["pool_grad"][n]
        assert np.abs(r32["pool_grad"][n] - ref).max() / np.abs(ref).max() < 1e-5
