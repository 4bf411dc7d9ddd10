"""Seeded synthetic workloads shaped like the paper's 182M-978M LLaMA-style MoE runs.

This module only draws random numbers and rounds them; it holds none of the
method's arithmetic, so the CUDA path and the CPU oracle can both be fed from
it.  The token values stand in for a training micro-batch (the paper trains on
16 x 1024-token micro-batches, App. D): only shapes matter to the MoE layer.

Recipe: x_0 ~ N(0,1) [T,d]; every expert and router weight ~ N(0, 0.02^2) (the down projection of
the 24-layer workloads ~ N(0, 0.02^2 / (2 L)), see CONFIGS);
sigma_l = 1; upstream gradient ~ N(0,1) [T,d]; one numpy PCG64 stream per tensor,
derived from (seed, tensor tag, layer) - for the pool weights one stream per
(seed, tensor tag, expert), so that the experts of a large pool can be drawn side by
side on all host cores.  In bf16 mode every tensor is rounded to
a bf16-representable value once, here, and returned as float32, so that both
sides read identical numbers.  The skewed workload adds to layer l's logits the
bias  beta * (ln p(rank_l(i)) - mean_j ln p(j)),  p(r) ~ r^-1.1 (Zipf), rank_l a
seeded permutation.  The bias is centred because the NormRouter score is
max(0, z/||z||): unlike a softmax it is not invariant to a common shift of the
logits, and an all-negative bias would zero almost every gate.  beta = 0.4 is the
smallest multiple of 0.05 for which, at seed 0, every layer of the skewed workload
has at least one expert without tokens (and one expert that more than 5 % of the
tokens select).
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

# name -> shape.  E of the benchmark spec is the paper's pool size M.
# ``private`` > 0 selects the layer-private layout of Eq. 1: layer l owns pool
# experts [private*l, private*(l+1)) and its router has ``private`` outputs.
CONFIGS = {
    "tiny_fp32":      dict(L=4,  d=256,  f=512,  M=16,  k=2, T=512,   dtype="fp32", private=0, zipf_beta=0.0),
    "182m":           dict(L=12, d=768,  f=2048, M=96,  k=2, T=16384, dtype="bf16", private=0, zipf_beta=0.0),
    "182m_vanilla":   dict(L=12, d=768,  f=2048, M=96,  k=2, T=16384, dtype="bf16", private=8, zipf_beta=0.0),
    # the paper's own baseline (Sec. 5.1): 8 private experts per layer, top-1, softmax router
    "182m_vanilla_softmax": dict(L=12, d=768, f=2048, M=96, k=1, T=16384, dtype="bf16", private=8, zipf_beta=0.0,
                                 router="softmax"),
    "182m_pool40":    dict(L=12, d=768,  f=2048, M=40,  k=2, T=16384, dtype="bf16", private=0, zipf_beta=0.0),
    # 24 residual blocks without a normalisation layer between them: with W_down ~ N(0, 0.02^2) the
    # stream grows quadratically per block, overflows bf16 near block 20 and the routing collapses onto
    # two experts.  These workloads therefore draw W_down with the depth-scaled standard deviation
    # 0.02 / sqrt(2 L) that transformer frameworks apply to output projections.
    "978m":           dict(L=24, d=1536, f=4096, M=192, k=2, T=32768, dtype="bf16", private=0, zipf_beta=0.0,
                           scaled_down_init=True),
    "978m_pool128":   dict(L=24, d=1536, f=4096, M=128, k=2, T=32768, dtype="bf16", private=0, zipf_beta=0.0,
                           scaled_down_init=True),
    "978m_vanilla":   dict(L=24, d=1536, f=4096, M=192, k=2, T=32768, dtype="bf16", private=8, zipf_beta=0.0,
                           scaled_down_init=True),
    # a quarter of one 182m layer (same rows per expert, same tiles): small profiler captures
    "182m_slice":     dict(L=1,  d=768,  f=2048, M=24,  k=2, T=4096,  dtype="bf16", private=0, zipf_beta=0.0),
    # profiler cases of the 978m shapes: an eighth of one layer (same rows per expert and tiles), and one
    # layer's full token batch over an eighth of the pool (activations larger than the L2 cache)
    "978m_slice":     dict(L=1,  d=1536, f=4096, M=24,  k=2, T=4096,  dtype="bf16", private=0, zipf_beta=0.0),
    "978m_tokens":    dict(L=1,  d=1536, f=4096, M=24,  k=2, T=32768, dtype="bf16", private=0, zipf_beta=0.0),
    # one private layer of eight experts at a quarter of its tokens: groups of ~16 row tiles (the CTA-pair kernels)
    "978m_groups":    dict(L=1,  d=1536, f=4096, M=8,   k=2, T=8192,  dtype="bf16", private=0, zipf_beta=0.0),
    "fine_zipf":      dict(L=12, d=768,  f=512,  M=384, k=8, T=16384, dtype="bf16", private=0, zipf_beta=0.4),
}

EPS = 1e-6          # epsilon of Eq. 7 (the paper gives no value)
ALPHA = 1e-2        # balance-loss coefficient used at the 182M scale (App. D)
INIT_STD = 0.02
ZIPF_S = 1.1


def round_to_bf16(a):
    """Round float32 values to the nearest bf16-representable float32 (ties to even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def _rng(seed, tag, layer=0):
    return np.random.default_rng([int(seed), int(tag), int(layer)])


def _normal(seed, tag, layer, shape, std, bf16):
    a = _rng(seed, tag, layer).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return round_to_bf16(a) if bf16 else a


def _pool_tensor(seed, tag, shape, std, bf16):
    """[M, rows, cols] pool weights, expert e from the stream (seed, tag, e); the experts are drawn,
    scaled and rounded by a pool of host threads (numpy releases the interpreter lock meanwhile)."""
    out = np.empty(shape, dtype=np.float32)

    def fill(e):
        out[e] = _normal(seed, tag, e, shape[1:], std, bf16)

    workers = min(len(os.sched_getaffinity(0)), shape[0]) if hasattr(os, "sched_getaffinity") else 1
    if workers <= 1:
        for e in range(shape[0]):
            fill(e)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, range(shape[0])))
    return out


def router_width(cfg):
    """Number of experts one router scores: M (shared pool), the private count, or M / G when the
    layers form ``groups`` = G sharing groups over depth."""
    if cfg.get("groups"):
        return cfg["M"] // cfg["groups"]
    return cfg["private"] if cfg["private"] else cfg["M"]


def expert_base(cfg, layer):
    """First pool expert visible to ``layer``'s router."""
    if cfg.get("groups"):
        return (layer // (cfg["L"] // cfg["groups"])) * (cfg["M"] // cfg["groups"])
    return cfg["private"] * layer if cfg["private"] else 0


def zipf_bias(cfg, layer, seed=0):
    """Additive logit bias of the skewed workload, or None."""
    beta = cfg.get("zipf_beta", 0.0)
    if not beta:
        return None
    m = router_width(cfg)
    ranks = np.arange(1, m + 1, dtype=np.float64)
    p = ranks ** (-ZIPF_S)
    p /= p.sum()
    perm = _rng(seed, 7, layer).permutation(m)          # expert i has rank perm[i]+1
    logp = np.log(p)
    return (beta * (logp[perm] - logp.mean())).astype(np.float32)


def make_inputs(cfg, seed=0, T=None, L=None):
    """Draw one workload.  ``T``/``L`` override the config (smaller parity cases).

    Returns dict(x0 [T,d], upstream [T,d], pool{W_gate [M,f,d], W_up [M,f,d],
    W_down [M,d,f]}, routers[l]{W_r [m,d], sigma, bias|None}) of float32 arrays.
    """
    T = cfg["T"] if T is None else T
    L = cfg["L"] if L is None else L
    d, f, M = cfg["d"], cfg["f"], cfg["M"]
    bf16 = cfg["dtype"] == "bf16"
    m = router_width(cfg)
    down_std = INIT_STD / float(np.sqrt(2.0 * cfg["L"])) if cfg.get("scaled_down_init") else INIT_STD
    pool = dict(
        W_gate=_pool_tensor(seed, 1, (M, f, d), INIT_STD, bf16),
        W_up=_pool_tensor(seed, 2, (M, f, d), INIT_STD, bf16),
        W_down=_pool_tensor(seed, 3, (M, d, f), down_std, bf16),
    )
    routers = []
    for l in range(L):
        routers.append(dict(W_r=_normal(seed, 4, l, (m, d), INIT_STD, bf16), sigma=1.0,
                            bias=zipf_bias(cfg, l, seed)))
    return dict(
        x0=_normal(seed, 5, 0, (T, d), 1.0, bf16),
        upstream=_normal(seed, 6, 0, (T, d), 1.0, bf16),
        pool=pool,
        routers=routers,
    )
