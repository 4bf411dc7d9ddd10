"""Shared helpers of the GPU parity tests: build a stack from a synthetic workload,
classify routing decisions by their margin, compare with the oracle."""
import numpy as np

from oracle import norm_router_c
from oracle import unipool_oracle as O
from paper_2605_06665_b200 import synth

MARGIN = 1e-4          # routing must be bit-exact where the k-th/(k+1)-th margin exceeds this

_C_CACHE = {}


def calib_c(m, k):
    """NormRouter constant for (experts scored, top-k): Alg. 1 with 20k draws, seed 0."""
    if (m, k) not in _C_CACHE:
        _C_CACHE[(m, k)] = float(np.float32(norm_router_c.estimate_c(m, k, 20_000, seed=0)))
    return _C_CACHE[(m, k)]


def f64(a):
    return np.asarray(a, dtype=np.float64)


def to_np(t):
    import torch
    if t.dtype == torch.bfloat16:
        t = t.float()
    return t.detach().cpu().numpy()


def rel_max(got, ref):
    """max|got - ref| / max|ref| (the norm of the parity bound)."""
    ref = f64(ref)
    den = np.abs(ref).max()
    num = np.abs(f64(got) - ref).max() if ref.size else 0.0
    return num / den if den > 0 else num


def _keys(z, mode):
    """What the top-k orders by, up to an increasing map: max(z, 0) for the NormRouter, z for softmax."""
    return f64(z) if mode == "softmax" else np.maximum(f64(z), 0.0)


def margin_safe(z, k, tol=MARGIN, mode="norm"):
    """Per token: is the top-k SET forced (k-th and (k+1)-th largest of max(z,0) differ
    by more than tol, or both are exactly zero scores with no logit within tol of 0),
    and is the slot ORDER forced (adjacent selected scores differ by more than tol)."""
    u = _keys(z, mode)
    srt = -np.sort(-u, axis=1)
    M = z.shape[1]
    if k < M:
        gap = srt[:, k - 1] - srt[:, k]
        near_zero = (np.abs(f64(z)) < tol).any(axis=1) & (mode != "softmax")
        set_safe = (gap > tol) | ((srt[:, k - 1] == 0) & ~near_zero)
        # zero-score picks are decided by index; they are safe only if no logit can flip sign
        set_safe &= ~((srt[:, k - 1] == 0) & near_zero)
        if mode == "softmax":                          # every key is a logit: only the gap decides
            set_safe = gap > tol
    else:
        set_safe = np.ones(z.shape[0], bool)
    if k > 1:
        adj = srt[:, :k - 1] - srt[:, 1:k]
        both_zero = (srt[:, :k - 1] == 0) & (srt[:, 1:k] == 0) & (mode != "softmax")
        order_safe = ((adj > tol) | both_zero).all(axis=1)
    else:
        order_safe = np.ones(z.shape[0], bool)
    return set_safe, order_safe & set_safe


def check_routing(idx_gpu, z_ref, idx_ref, k, mode="norm"):
    """Bit-exact where the margin forces the decision; a valid top-k elsewhere."""
    set_safe, order_safe = margin_safe(z_ref, k, mode=mode)
    assert (idx_gpu[order_safe] == idx_ref[order_safe]).all(), "routing differs on margin-safe tokens"
    only_set = set_safe & ~order_safe
    assert (np.sort(idx_gpu[only_set], axis=1) == np.sort(idx_ref[only_set], axis=1)).all()
    # everywhere: k distinct in-range experts whose scores are within tol of the true top-k
    M = z_ref.shape[1]
    assert ((idx_gpu >= 0) & (idx_gpu < M)).all()
    srt = np.sort(idx_gpu, axis=1)
    assert (srt[:, 1:] != srt[:, :-1]).all() if k > 1 else True
    u = _keys(z_ref, mode)
    kth = -np.sort(-u, axis=1)[:, k - 1]
    picked = np.take_along_axis(u, idx_gpu.astype(np.int64), axis=1)
    assert (picked >= kth[:, None] - MARGIN).all()
    return set_safe, order_safe


def build_stack(cfg, inputs, T=None, L=None, deferred_wgrad=False, c=None):
    from paper_2605_06665_b200.stack import UniPoolStack
    T = cfg["T"] if T is None else T
    L = cfg["L"] if L is None else L
    m = synth.router_width(cfg)
    c = calib_c(m, cfg["k"]) if c is None else c
    st = UniPoolStack(L, cfg["d"], cfg["f"], cfg["M"], cfg["k"], T, cfg["dtype"], cfg["private"], c=c,
                      eps=synth.EPS, alpha=synth.ALPHA, deferred_wgrad=deferred_wgrad, groups=cfg.get("groups"),
                      router=cfg.get("router", "norm"))
    st.load(inputs["pool"], inputs["routers"][:L])
    return st


def oracle_params(inputs, L, mode="norm"):
    pool = {n: f64(w) for n, w in inputs["pool"].items()}
    routers = [dict(W_r=f64(r["W_r"]), sigma=float(r["sigma"]), mode=mode,
                    bias=None if r["bias"] is None else f64(r["bias"])) for r in inputs["routers"][:L]]
    return pool, routers
