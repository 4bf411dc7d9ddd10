"""Per-token, per-slot statement of the UniPool forward pass in plain Python.

TEST INFRASTRUCTURE ONLY.  Scalars are Python floats (IEEE double), containers
are nested lists, loops are explicit; there is no numpy in the arithmetic.  It
exists to pin ``unipool_oracle`` on tiny inputs: a wrong axis, a transposed
operand or a dropped term in the vectorised code shows up as a mismatch here.
"""
from __future__ import annotations

import math


def _dot(a, b):
    acc = 0.0
    for p, q in zip(a, b):
        acc += p * q
    return acc


def norm_router_token(h, W_r, sigma, c, eps, bias=None):
    """Eq. 7 for one token: z = W_r h, s_i = sigma*c*max(0, z_i/(||z||_2+eps))."""
    z = [_dot(row, h) + (0.0 if bias is None else bias[i]) for i, row in enumerate(W_r)]
    n = math.sqrt(sum(v * v for v in z))
    s = [sigma * c * max(0.0, v / (n + eps)) for v in z]
    return z, n, s


def top_k_token(s, k):
    """k highest scores, ties to the lowest index, by repeated scan (Sec. 4.3)."""
    chosen = []
    for _ in range(k):
        best = -1
        for i, v in enumerate(s):
            if i in chosen:
                continue
            if best < 0 or v > s[best]:      # strict '>' keeps the lowest index on ties
                best = i
        chosen.append(best)
    return chosen


def swiglu_expert_token(h, W_gate, W_up, W_down):
    """e(h) = W_down (silu(W_gate h) * (W_up h)) for one token."""
    a = []
    for wg, wu in zip(W_gate, W_up):
        gg = _dot(wg, h)
        uu = _dot(wu, h)
        a.append(gg / (1.0 + math.exp(-gg)) * uu)
    return [_dot(wd, a) for wd in W_down]


def stack_forward(x0, routers, pool, k, c, eps, views=None):
    """x_{l+1} = x_l + sum_{i in top-k} g_{l,i} e_i(x_l)  (Eq. 2 in a residual stack).

    x0: list of T token vectors.  routers: list of dicts(W_r, sigma, bias?).
    pool: dict(W_gate, W_up, W_down) of nested lists.  Returns per layer:
    dict(idx, g, counts, S, x_next).
    """
    out = []
    x = [list(row) for row in x0]
    for l, router in enumerate(routers):
        base = 0 if views is None else views[l]
        M = len(router["W_r"])
        counts = [0] * M
        S = [0.0] * M
        idx_l, g_l, x_next = [], [], []
        for h in x:
            _, _, s = norm_router_token(h, router["W_r"], router["sigma"], c, eps, router.get("bias"))
            for i in range(M):
                S[i] += s[i]
            sel = top_k_token(s, k)
            y = [0.0] * len(h)
            for i in sel:
                counts[i] += 1
                e = swiglu_expert_token(h, pool["W_gate"][base + i], pool["W_up"][base + i],
                                        pool["W_down"][base + i])
                for q in range(len(h)):
                    y[q] += s[i] * e[q]
            idx_l.append(sel)
            g_l.append([s[i] for i in sel])
            x_next.append([h[q] + y[q] for q in range(len(h))])
        out.append(dict(idx=idx_l, g=g_l, counts=counts, S=S, x_next=x_next))
        x = x_next
    return out


def pool_aux_loss(counts, S, T, k, alpha):
    """Eq. 5 written out: alpha*M*sum_i [mean_l counts/(T k)] * [mean_l S/T]."""
    L = len(counts)
    M = len(counts[0])
    total = 0.0
    for i in range(M):
        fbar = sum(counts[l][i] / (T * k) for l in range(L)) / L
        pbar = sum(S[l][i] / T for l in range(L)) / L
        total += fbar * pbar
    return alpha * M * total
