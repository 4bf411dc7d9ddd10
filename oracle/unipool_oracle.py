"""Plain numpy oracle of the UniPool MoE layer: forward, balance loss, backward.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Every function states
the passage of the paper it follows.  There is no blocking, fusion or
reordering: a reader can check each line against the equation it cites.

Notation (the paper's): L layers, M pool experts, k experts per token, d model
width, f expert width, T tokens, z = W_r h router logits, s NormRouter scores,
g gates, f_i^(l) token fraction, P_i^(l) mean score, sigma learnable router
scale, c fixed calibration constant, alpha balance coefficient.

Every function takes ``dtype`` from its inputs: feed float64 arrays for the
reference-grade result, float32 arrays for the fp32 mode.

Readings taken where the paper is silent (each is a plain-language statement,
none changes an equation):
  * gates are the selected scores themselves, not renormalised over the top-k
    (Eq. 2 uses g_{l,i}; c exists to give the unnormalised scores unit scale);
  * top-k is taken on the scores s (Sec. 4.3), key = (score descending, expert
    index ascending), so ties - including ties at score 0 - go to the lowest
    index;
  * the norm in Eq. 7 is over the whole logit vector z, eps is added to it;
  * f_i^(l) = (#assignments to i) / (T k) so that sum_i f_i = 1 for any k;
  * P_i^(l) is the mean over tokens of the full score vector (all M entries);
  * the expert is a bias-free SwiGLU FFN, silu on the "gate" projection;
  * no token is dropped: every (token, slot) assignment is computed;
  * only P carries gradient in the balance loss; f-bar is a constant (App. G).
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# NormRouter, Eq. 7, and top-k selection, Sec. 4.3
# --------------------------------------------------------------------------
def router_logits(x, W_r, bias=None):
    """z = W_r h for every token (Sec. 4.3, sentence before Eq. 7).

    x [T,d], W_r [M,d] -> z [T,M].  ``bias`` [M] is an optional additive logit
    offset (used only to skew the synthetic load; not part of the paper).
    """
    z = x @ W_r.T
    if bias is not None:
        z = z + bias[None, :]
    return z


def norm_router_scores(z, sigma, c, eps):
    """Eq. 7: s_i = sigma * c * max(0, z_i / (||z||_2 + eps)).

    Returns (s [T,M], n [T]) with n the L2 norm of the whole logit vector.
    """
    n = np.sqrt(np.sum(z * z, axis=-1))
    s = sigma * c * np.maximum(0.0, z / (n[:, None] + eps))
    return s.astype(z.dtype), n.astype(z.dtype)


def softmax_router_scores(z):
    """The conventional router the paper compares against (Sec. 4.3, first sentence; the vanilla
    baseline of Sec. 5.1): s_i = exp(z_i) / sum_j exp(z_j) over the router's experts.

    Returns (s [T,M], lse [T]) with lse = log sum_j exp(z_j); the largest logit is subtracted before
    exponentiation, which changes nothing in exact arithmetic.
    """
    m = np.max(z, axis=-1)
    e = np.exp(z - m[:, None])
    tot = np.sum(e, axis=-1)
    s = e / tot[:, None]
    return s.astype(z.dtype), (m + np.log(tot)).astype(z.dtype)


def top_k(s, k):
    """Indices of the k highest scores per token (Sec. 4.3, "Top-k selection"),
    descending score, ties broken by the lowest expert index.  s [T,M] -> idx [T,k] int32.
    """
    # a stable sort of the negated scores keeps equal scores in index order
    order = np.argsort(-s, axis=-1, kind="stable")
    return order[:, :k].astype(np.int32)


def route(x, W_r, sigma, c, eps, k, bias=None, forced_idx=None, mode="norm"):
    """One layer's router: logits, scores (Eq. 7, or softmax with ``mode="softmax"``, where sigma, c
    and eps play no part and ``n`` holds log-sum-exp of the logits), top-k, gates and statistics.

    Returns a dict with
      z [T,M], n [T], s [T,M], idx [T,k] int32, g [T,k] (g = s at idx, Eq. 2),
      counts [M] int64 (#assignments per expert), S [M] (sum_t s_{t,i}, the
      numerator of P_i in Eq. 3 with scores in place of probabilities).
    ``forced_idx`` replaces the top-k decision (used by tests to hold routing
    fixed); gates are still read from s.
    """
    z = router_logits(x, W_r, bias)
    if mode == "softmax":
        s, n = softmax_router_scores(z)
    else:
        assert mode == "norm", mode
        s, n = norm_router_scores(z, sigma, c, eps)
    idx = top_k(s, k) if forced_idx is None else np.asarray(forced_idx, dtype=np.int32)
    g = np.take_along_axis(s, idx.astype(np.int64), axis=1)
    M = W_r.shape[0]
    counts = np.bincount(idx.reshape(-1), minlength=M).astype(np.int64)
    S = s.sum(axis=0)
    return dict(z=z, n=n, s=s, idx=idx, g=g, counts=counts, S=S)


# --------------------------------------------------------------------------
# expert-contiguous permutation (the grouped layout a grouped GEMM consumes)
# --------------------------------------------------------------------------
def dispatch_map(idx, M, row_align=1):
    """Stable expert-major ordering of the T*k assignments.

    The paper only says experts run as a grouped GEMM (Table 7); the map is the
    plain definition of "sort assignments by expert, keep token-major order
    inside an expert".  Group e occupies rows offsets[e] .. offsets[e]+counts[e];
    each group's start is rounded up to ``row_align`` rows (pad rows hold zeros).

    Returns offsets [M+1] int64, row_of [T,k] int64, token_of [offsets[M]]
    int64 (-1 on pad rows).
    """
    T, k = idx.shape
    counts = np.bincount(idx.reshape(-1), minlength=M)
    padded = (counts + row_align - 1) // row_align * row_align
    offsets = np.zeros(M + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(padded)
    row_of = np.empty((T, k), dtype=np.int64)
    token_of = np.full(int(offsets[M]), -1, dtype=np.int64)
    fill = offsets[:-1].copy()
    for t in range(T):            # token-major, then slot order
        for j in range(k):
            e = int(idx[t, j])
            row_of[t, j] = fill[e]
            token_of[fill[e]] = t
            fill[e] += 1
    return offsets, row_of, token_of


# --------------------------------------------------------------------------
# SwiGLU expert and the layer output, Eq. 2
# --------------------------------------------------------------------------
def silu(a):
    """silu(a) = a / (1 + exp(-a))."""
    return a / (1.0 + np.exp(-a))


def silu_grad(a):
    """d silu / da = sig(a) * (1 + a * (1 - sig(a))), sig the logistic function."""
    sig = 1.0 / (1.0 + np.exp(-a))
    return sig * (1.0 + a * (1.0 - sig))


def expert_ffn(h, W_gate_e, W_up_e, W_down_e):
    """e_i(h) = W_down (silu(W_gate h) * (W_up h)) for a batch of rows h [r,d]
    (LLaMA-style SwiGLU FFN, App. B / Table 8).  Returns (G, U, A, Y).
    """
    G = h @ W_gate_e.T
    U = h @ W_up_e.T
    A = silu(G) * U
    Y = A @ W_down_e.T
    return G, U, A, Y


def moe_layer_output(x, idx, g, pool, expert_base=0, tokens=None):
    """Eq. 2: FFN_l(x_t) = sum_j g_{t,j} * e_{idx_{t,j}}(x_t).

    ``pool`` = dict(W_gate [M,f,d], W_up [M,f,d], W_down [M,d,f]).  Router index i
    addresses pool expert ``expert_base + i`` (UniPool: base 0 for every layer;
    the layer-private layout of Eq. 1: base = first private expert of the layer).
    ``tokens`` restricts the evaluation to a list of token ids (result has one
    row per listed token); each token's value is independent of the others.
    """
    tok = np.arange(x.shape[0]) if tokens is None else np.asarray(tokens)
    y = np.zeros((len(tok), x.shape[1]), dtype=x.dtype)
    sub_idx = idx[tok]
    sub_g = g[tok]
    for e in np.unique(sub_idx):
        rows, slots = np.nonzero(sub_idx == e)
        pe = expert_base + int(e)
        _, _, _, Y = expert_ffn(x[tok[rows]], pool["W_gate"][pe], pool["W_up"][pe], pool["W_down"][pe])
        np.add.at(y, rows, sub_g[rows, slots][:, None] * Y)
    return y


def layer_forward(x, router, pool, k, c, eps, expert_base=0, forced_idx=None):
    """One residual MoE block: route, Eq. 2, x_next = x + FFN_l(x)."""
    r = route(x, router["W_r"], router["sigma"], c, eps, k, router.get("bias"), forced_idx,
              router.get("mode", "norm"))
    y = moe_layer_output(x, r["idx"], r["g"], pool, expert_base)
    r["y"] = y
    r["x"] = x
    r["x_next"] = x + y
    return r


def stack_forward(x0, routers, pool, k, c, eps, views=None, forced_idx=None):
    """L residual MoE blocks over one pool.  ``views[l] = expert_base`` of layer l
    (None: every layer sees the pool from expert 0 - UniPool).  Returns the list
    of per-layer caches; cache[-1]["x_next"] is x_L.
    """
    caches = []
    x = x0
    for l, router in enumerate(routers):
        base = 0 if views is None else views[l]
        fi = None if forced_idx is None else forced_idx[l]
        cache = layer_forward(x, router, pool, k, c, eps, base, fi)
        caches.append(cache)
        x = cache["x_next"]
    return caches


# --------------------------------------------------------------------------
# balance losses, Eqs. 3-6
# --------------------------------------------------------------------------
def layer_fractions(counts, S, T, k):
    """f_i^(l) = counts_i / (T k);  P_i^(l) = S_i / T  (definitions under Eq. 3)."""
    f = counts.astype(S.dtype) / (T * k)
    P = S / T
    return f, P


def pool_aux_loss(counts, S, T, k, alpha, fbar_prev=None):
    """Eq. 4 and Eq. 5: fbar_i = mean_l f_i^(l), Pbar_i = mean_l P_i^(l),
    L_pool = alpha * M * sum_i fbar_i * Pbar_i.

    counts [L,M] int, S [L,M].  ``fbar_prev`` (App. G, one-step-behind) replaces
    fbar in the loss.  Returns (loss, fbar_of_this_batch [M], coef [M]) where
    coef_i = alpha*M*fbar_i/(L*T) is dL_pool/ds^(l)_{t,i} for every t and l
    (only P carries gradient).
    """
    L, M = counts.shape
    f = np.stack([layer_fractions(counts[l], S[l], T, k)[0] for l in range(L)])
    P = np.stack([layer_fractions(counts[l], S[l], T, k)[1] for l in range(L)])
    fbar = f.mean(axis=0)
    Pbar = P.mean(axis=0)
    f_used = fbar if fbar_prev is None else np.asarray(fbar_prev, dtype=S.dtype)
    loss = alpha * M * np.sum(f_used * Pbar)
    coef = alpha * M * f_used / (L * T)
    return loss, fbar, coef


def pool_aux_loss_decomposed(counts, S, T, k, alpha):
    """Eq. 6: (1/L) sum_l alpha*M*sum_i fbar_i P_i^(l) - the per-layer form."""
    L, M = counts.shape
    f = np.stack([layer_fractions(counts[l], S[l], T, k)[0] for l in range(L)])
    fbar = f.mean(axis=0)
    total = 0.0
    for l in range(L):
        _, P_l = layer_fractions(counts[l], S[l], T, k)
        total += alpha * M * np.sum(fbar * P_l)
    return total / L


def switch_aux_loss(counts_l, S_l, T, k, alpha):
    """Eq. 3 for one layer with E private experts: alpha * E * sum_i f_i P_i."""
    E = counts_l.shape[0]
    f, P = layer_fractions(counts_l, S_l, T, k)
    return alpha * E * np.sum(f * P)


# --------------------------------------------------------------------------
# backward: derivatives of Eq. 2 and Eq. 7
# --------------------------------------------------------------------------
def expert_path_backward(x, idx, g, pool, dy, expert_base=0, pool_grad=None, tokens=None,
                         experts=None):
    """Derivative of y_t = sum_j g_{t,j} e_{idx_{t,j}}(x_t) given dy = dJ/dy.

    Returns (dx_expert [T,d], dg [T,k]) and adds the weight gradients into
    ``pool_grad`` (same keys/shapes as ``pool``; the SAME arrays for every layer
    that calls this - each shared expert accumulates gradient from all L layers,
    Sec. 3).  For row h of expert e with incoming dY = g * dy_t:
        dg      = <dy_t, Y>
        dA      = W_down^T dY                dW_down += dY A^T
        dG      = dA * U * silu'(G)          dW_gate += dG h^T
        dU      = dA * silu(G)               dW_up   += dU h^T
        dh      = W_gate^T dG + W_up^T dU
    ``tokens``: evaluate dx, dg only for these tokens (rows of the result follow
    the list; weight gradients are then NOT accumulated).  ``experts``: accumulate
    weight gradients only for these router-local expert ids (over all tokens).
    """
    tok = np.arange(x.shape[0]) if tokens is None else np.asarray(tokens)
    sub_idx = idx[tok]
    sub_g = g[tok]
    dx = np.zeros((len(tok), x.shape[1]), dtype=x.dtype)
    dg = np.zeros(sub_g.shape, dtype=x.dtype)
    todo = np.unique(sub_idx) if experts is None else np.asarray(experts)
    for e in todo:
        rows, slots = np.nonzero(sub_idx == e)
        if rows.size == 0:
            continue
        pe = expert_base + int(e)
        Wg, Wu, Wd = pool["W_gate"][pe], pool["W_up"][pe], pool["W_down"][pe]
        h = x[tok[rows]]
        G, U, A, Y = expert_ffn(h, Wg, Wu, Wd)
        dy_rows = dy[tok[rows]]
        dg[rows, slots] = np.sum(dy_rows * Y, axis=1)
        dY = sub_g[rows, slots][:, None] * dy_rows
        dA = dY @ Wd
        dG = dA * U * silu_grad(G)
        dU = dA * silu(G)
        np.add.at(dx, rows, dG @ Wg + dU @ Wu)
        if pool_grad is not None and tokens is None:
            pool_grad["W_down"][pe] += dY.T @ A
            pool_grad["W_gate"][pe] += dG.T @ h
            pool_grad["W_up"][pe] += dU.T @ h
    return dx, dg


def route_backward(x, W_r, sigma, c, eps, z, n, idx, dg, coef=None, mode="norm"):
    """Derivative of the score function followed by z = W_r x.

    ``mode="softmax"``: s = softmax(z), so with q_t = sum_i ds_{t,i} s_{t,i}
        dz_{t,m} = s_{t,m} (ds_{t,m} - q_t),   dsigma = 0   (``n`` is not used).
    ``mode="norm"`` (Eq. 7):

    ds_{t,i} = coef_i + sum_{j: idx_{t,j}=i} dg_{t,j}   (coef: balance-loss term)
    With u = max(z,0) and q_t = sum_i ds_{t,i} u_{t,i}:
        dz_{t,m} = sigma c [ 1{z_m>0} ds_m / (n+eps) - z_m q_t / (n (n+eps)^2) ]
    (rows with n = 0 have dz = 0),  dsigma = c sum ds u / (n+eps),
    dW_r = dz^T x,  dx_router = dz W_r.
    Returns dict(dz, dW_r, dsigma, dx).
    """
    T, M = z.shape
    ds = np.zeros((T, M), dtype=z.dtype)
    if coef is not None:
        ds += np.asarray(coef, dtype=z.dtype)[None, :]
    np.add.at(ds, (np.repeat(np.arange(T), idx.shape[1]), idx.reshape(-1).astype(np.int64)),
              dg.reshape(-1))
    if mode == "softmax":
        sm, _ = softmax_router_scores(z)
        q = np.sum(ds * sm, axis=1)
        dz = (sm * (ds - q[:, None])).astype(z.dtype)
        return dict(dz=dz, dW_r=dz.T @ x, dsigma=z.dtype.type(0), dx=dz @ W_r, ds=ds)
    assert mode == "norm", mode
    u = np.maximum(z, 0.0)
    q = np.sum(ds * u, axis=1)
    ne = n + eps
    safe_n = np.where(n > 0, n, 1.0)
    dz = sigma * c * ((z > 0) * ds / ne[:, None] - z * (q / (safe_n * ne * ne))[:, None])
    dz = np.where((n > 0)[:, None], dz, 0.0).astype(z.dtype)
    dsigma = c * np.sum(ds * u / ne[:, None])
    return dict(dz=dz, dW_r=dz.T @ x, dsigma=dsigma, dx=dz @ W_r, ds=ds)


def layer_backward(cache, router, pool, k, c, eps, dx_next, coef, pool_grad, expert_base=0):
    """Backward of x_next = x + FFN_l(x) (and of this layer's share of the balance
    loss through ``coef``).  Returns dict(dx, dW_r, dsigma, dg)."""
    x = cache["x"]
    dx_e, dg = expert_path_backward(x, cache["idx"], cache["g"], pool, dx_next, expert_base, pool_grad)
    rb = route_backward(x, router["W_r"], router["sigma"], c, eps, cache["z"], cache["n"],
                        cache["idx"], dg, coef, router.get("mode", "norm"))
    return dict(dx=dx_next + dx_e + rb["dx"], dW_r=rb["dW_r"], dsigma=rb["dsigma"], dg=dg,
                dx_expert=dx_e, dx_router=rb["dx"])


def unique_experts(idx_layers, views=None):
    """App. E: U(x) = |{ e_l(x) : l = 1..L }| per token - the number of distinct pool experts the
    token selects over all layers (every one of the k picks of a layer counts).  ``idx_layers`` is a
    list of [T,k] index arrays, ``views[l]`` the first pool expert of layer l (None: shared pool)."""
    L = len(idx_layers)
    T = idx_layers[0].shape[0]
    out = np.zeros(T, dtype=np.int64)
    for t in range(T):
        seen = set()
        for l in range(L):
            base = 0 if views is None else views[l]
            for e in idx_layers[l][t]:
                seen.add(base + int(e))
        out[t] = len(seen)
    return out


def zeros_like_pool(pool):
    return {name: np.zeros_like(w) for name, w in pool.items()}


def stack_objective_and_grads(x0, routers, pool, k, c, eps, alpha, upstream, views=None,
                              forced_idx=None, fbar_prev=None, n_view=None, aux_groups=None,
                              replica_stats=None):
    """J = sum(upstream * x_L) + balance loss, and dJ/d(everything).

    UniPool (views None): balance loss = Eq. 5 over all L layers.  Layer-private
    layout (views given, each layer owning ``n_view`` experts): balance loss =
    sum_l Eq. 3.  Sharing scope G (Sec. 5.3 ablation: G pools over depth): ``aux_groups`` lists the
    layers of every group; each group is a pool of its own, so its balance loss is Eq. 5 over the
    group's layers and experts (G = L gives sum_l Eq. 3, G = 1 gives Eq. 5).
    Routing decisions and f-bar are constants of the derivative.
    Data-parallel replicas (App. D trains data parallel; the batch of Eqs. 3-5 is then the union of
    the replicas' tokens): ``replica_stats(counts, S) -> (counts, S, T)`` returns the statistics summed
    over all replicas and the total token count; the balance loss returned is the whole batch's, the
    gradients are this replica's share (their sum over replicas is the whole batch's gradient).
    Returns dict(J, loss_aux, caches, pool_grad, router_grads [L], dx0).
    """
    L = len(routers)
    T = x0.shape[0]
    caches = stack_forward(x0, routers, pool, k, c, eps, views, forced_idx)
    counts = np.stack([cch["counts"] for cch in caches])
    S = np.stack([cch["S"] for cch in caches])
    if replica_stats is not None:
        counts, S, T = replica_stats(counts, S)
    if aux_groups is not None:
        loss_aux = 0.0
        coefs = [None] * L
        for layers in aux_groups:
            lo, _, co = pool_aux_loss(counts[layers], S[layers], T, k, alpha)
            loss_aux += lo
            for l in layers:
                coefs[l] = co
    elif views is None:
        loss_aux, fbar, coef = pool_aux_loss(counts, S, T, k, alpha, fbar_prev)
        coefs = [coef] * L
    else:
        loss_aux = 0.0
        coefs = []
        for l in range(L):
            lo, _, co = pool_aux_loss(counts[l:l + 1], S[l:l + 1], T, k, alpha)
            loss_aux += lo
            coefs.append(co)
    x_L = caches[-1]["x_next"]
    J = np.sum(upstream * x_L) + loss_aux
    pool_grad = zeros_like_pool(pool)
    router_grads = [None] * L
    dx = upstream.astype(x0.dtype)
    for l in reversed(range(L)):
        base = 0 if views is None else views[l]
        out = layer_backward(caches[l], routers[l], pool, k, c, eps, dx, coefs[l], pool_grad, base)
        router_grads[l] = dict(dW_r=out["dW_r"], dsigma=out["dsigma"], dg=out["dg"],
                               dx_expert=out["dx_expert"], dx_router=out["dx_router"], dx=out["dx"])
        dx = out["dx"]
    return dict(J=J, loss_aux=loss_aux, caches=caches, pool_grad=pool_grad,
                router_grads=router_grads, dx0=dx, counts=counts, S=S, coefs=coefs)
