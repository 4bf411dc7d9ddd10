"""Monte-Carlo estimate of the NormRouter calibration constant c (Alg. 1, App. H).

TEST INFRASTRUCTURE ONLY.

c = E[ 1 / || top-k( ReLU(x / ||x||_2) ) ||_2 ],  x ~ N(0, I_E).

The algorithm does not say what to do with a draw that has no positive
component (its top-k norm is 0); such a draw has probability 2^-E and is
skipped here, i.e. the expectation is conditioned on at least one positive
component.  c only scales the scores; both the oracle and the CUDA library take
it as an input number, so its value never enters a parity comparison.
"""
from __future__ import annotations

import numpy as np


def topk_norm(x, k):
    """|| top-k( ReLU(x / ||x||_2) ) ||_2 for each row of x [m,E] (Alg. 1, App. H)."""
    y = np.maximum(x / np.linalg.norm(x, axis=1, keepdims=True), 0.0)
    y_sorted = -np.sort(-y, axis=1)               # descending
    top = y_sorted[:, :k]
    return np.sqrt(np.sum(top * top, axis=1))


def estimate_c(E, k, n_samples=100_000, seed=0):
    """Run Alg. 1 with ``n_samples`` draws; returns a Python float."""
    rng = np.random.default_rng(seed)
    total = 0.0
    used = 0
    chunk = 8192
    done = 0
    while done < n_samples:
        m = min(chunk, n_samples - done)
        nrm = topk_norm(rng.standard_normal((m, E)), k)
        ok = nrm > 0
        total += float(np.sum(1.0 / nrm[ok]))
        used += int(ok.sum())
        done += m
    return total / used
