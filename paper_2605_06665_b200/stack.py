"""A residual stack of UniPool MoE layers driven through the C-ABI library.

``UniPoolStack`` owns the device buffers (PyTorch tensors) and issues, per layer,
the library calls route -> dispatch -> expert_fwd -> combine (forward), then
pool_aux_loss, then expert_bwd -> route_bwd per layer in reverse (backward).
It contains no arithmetic of its own: every tensor it returns was written by a
CUDA kernel of the library.

Layer l computes x_{l+1} = x_l + sum_{i in top-k} g_{l,i}(x_l) e_i(x_l)  (Eq. 2),
all layers sharing one pool of experts; with ``private = E`` layer l instead
owns pool experts [E*l, E*(l+1)) (the layer-private layout of Eq. 1); with
``groups = G`` (sharing scope of the ablation in Sec. 5.3) the L layers form G
consecutive groups of L/G layers, group g sharing pool experts [g*M/G, (g+1)*M/G)
with its own balance loss (Eq. 5 over the group's layers; G = 1 is UniPool, G = L
the private layout).  In the private layout the
balance loss is the per-layer loss of Eq. 3 summed over layers.  ``router="softmax"``
replaces the NormRouter of Eq. 7 by the conventional softmax router of the paper's
baselines (Sec. 5.1) in every layer.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class UniPoolStack:
    def __init__(self, L, d, f, M, k, T, dtype="bf16", private=0, c=1.0, eps=1e-6, alpha=1e-2,
                 device="cuda", deferred_wgrad=False, recompute=False, groups=None, router="norm"):
        self.L, self.d, self.f, self.M, self.k, self.T = L, d, f, M, k, T
        if groups is None:
            groups = L if private else 1
        if L % groups or M % groups or (private and (groups != L or private * L != M)):
            raise ValueError("layers and pool experts must split evenly into the sharing groups")
        self.G, self.Lg = groups, L // groups              # sharing groups over depth, layers per group
        self.private = private
        self.m = M // groups                               # experts one router scores
        self.alpha = alpha
        self.c, self.eps = c, eps
        # recompute: keep only x_l and the routing state of a layer; its permuted activations are
        # rebuilt in backward (MoE-layer activation recompute, App. D), so the weight gradient is
        # taken layer by layer
        self.recompute = recompute
        self.deferred_wgrad = deferred_wgrad and self.Lg > 1 and not recompute
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if dtype == "bf16" else torch.float32
        if router not in ("norm", "softmax"):
            raise ValueError("router must be 'norm' or 'softmax'")
        self.router = router
        self.cfg = B.make_config(d, f, M, k, L, T, B.BF16 if dtype == "bf16" else B.FP32, eps, c,
                                 B.ROUTER_SOFTMAX if router == "softmax" else B.ROUTER_NORM)
        self.ctx = B.Context(self.cfg, self.device)
        cap = self.ctx.row_capacity
        self.cap = cap
        dev, td = self.device, self.tdtype
        i32, f32 = torch.int32, torch.float32
        e = lambda *shape, dtype=td: torch.empty(*shape, dtype=dtype, device=dev)
        # parameters
        self.W_gu = e(M, 2 * f, d)
        self.W_down = e(M, d, f)
        self.W_r = e(L, self.m, d, dtype=f32)
        self.sigma = [1.0] * L
        self.bias = None                                   # [L, m] float or None
        # gradients (fp32; one buffer per pool expert, shared by all layers)
        self.dW_gu = torch.zeros(M, 2 * f, d, dtype=f32, device=dev)
        self.dW_down = torch.zeros(M, d, f, dtype=f32, device=dev)
        self.dW_r = torch.zeros(L, self.m, d, dtype=f32, device=dev)
        self.dsigma = torch.zeros(L, dtype=f32, device=dev)
        # activations and routing state kept for backward
        self.x = e(L + 1, T, d)
        self.idx = e(L, T, k, dtype=i32)
        self.gate = e(L, T, k, dtype=f32)
        self.counts = e(L, self.m, dtype=i32)
        self.score_sum = e(L, self.m, dtype=f32)
        self.znorm = e(L, T, dtype=f32)
        self.z = e(L, T, self.m, dtype=f32)
        self.offsets = e(L, self.m + 1, dtype=i32)
        self.row_of = e(L, T, k, dtype=i32)
        self.token_of = e(L, cap, dtype=i32)
        self.tile_expert = e(L, cap // B.ROW_ALIGN, dtype=i32)
        ns = 1 if recompute else L                         # layers whose permuted activations are kept
        self.Xp = e(ns, cap, d)
        self.GU = e(ns, cap, 2 * f)
        self.A = e(ns, cap, f)
        self.Yp = e(ns, cap, d)
        nb = L if self.deferred_wgrad else 1
        self.dYp = e(nb, cap, d)
        self.dGU = e(nb, cap, 2 * f)
        self.dx = e(2, T, d)                               # ping-pong dx_{l+1} -> dx_l
        self.dgate = e(T, k, dtype=f32)
        # balance loss
        n_aux = groups                                     # one balance loss per sharing group
        self.loss = torch.zeros(n_aux, dtype=f32, device=dev)
        self.coef = e(n_aux, self.m, dtype=f32)
        self.fbar = e(n_aux, self.m, dtype=f32)
        self.fbar_lag = None                               # f-bar of the previous micro-batch (App. G)
        self._copy_stream = None                           # host <-> device copies beside the compute

    # ------------------------------------------------------------------ parameters
    def load(self, pool, routers):
        """pool: dict(W_gate [M,f,d], W_up [M,f,d], W_down [M,d,f]); routers: list of
        dict(W_r [m,d], sigma, bias|None) - numpy float32 arrays (host)."""
        f = self.f
        self.W_gu[:, :f].copy_(torch.from_numpy(pool["W_gate"]))
        self.W_gu[:, f:].copy_(torch.from_numpy(pool["W_up"]))
        self.W_down.copy_(torch.from_numpy(pool["W_down"]))
        for l, r in enumerate(routers):
            self.W_r[l].copy_(torch.from_numpy(r["W_r"]))
            self.sigma[l] = float(r["sigma"])
        if routers[0].get("bias") is not None:
            self.bias = torch.from_numpy(np.stack([r["bias"] for r in routers])).to(self.device)
        self.ctx.router_prepare(None, 0, self.m)           # forget router terms formed from older weights
        torch.cuda.synchronize(self.device)

    def base(self, l):
        return (l // self.Lg) * self.m

    def slot(self, l):
        """Index of layer l's permuted activations (one shared slot when they are recomputed)."""
        return 0 if self.recompute else l

    def zero_grad(self):
        self.dW_gu.zero_(); self.dW_down.zero_(); self.dW_r.zero_(); self.dsigma.zero_()

    def zero_router_grad(self):
        self.dW_r.zero_(); self.dsigma.zero_()

    # ------------------------------------------------------------------ forward
    def forward_layer(self, l, T=None):
        T = self.T if T is None else T
        c = self.ctx
        bias = None if self.bias is None else self.bias[l]
        c.route(self.x[l], T, self.W_r[l], self.sigma[l], bias, self.m, self.idx[l], self.gate[l],
                self.counts[l], self.score_sum[l], self.znorm[l], self.z[l])
        self.permute_and_experts(l, T)
        c.combine(self.Yp[self.slot(l)], self.row_of[l], self.gate[l], T, self.x[l], self.x[l + 1])

    def permute_and_experts(self, l, T):
        """dispatch + expert forward of layer l from x_l and its routing decision (also the
        recompute step of backward)."""
        c, s = self.ctx, self.slot(l)
        c.dispatch(self.x[l], T, self.idx[l], self.m, self.offsets[l], self.row_of[l], self.token_of[l],
                   self.tile_expert[l], self.Xp[s])
        c.expert_fwd(self.Xp[s], self.offsets[l], self.tile_expert[l], self.W_gu, self.W_down,
                     self.base(l), self.m, self.GU[s], self.A[s], self.Yp[s])

    def forward(self, x0=None, T=None):
        T = self.T if T is None else T
        if x0 is not None:
            self.x[0, :T].copy_(x0, non_blocking=True)
        # the routers' weights may have changed since the last pass: one kernel re-forms the bf16 terms
        # of all layers (used by this forward pass and by the backward pass that follows it)
        self.ctx.router_prepare(self.W_r, self.L, self.m)
        for l in range(self.L):
            self.forward_layer(l, T)
        return self.x[self.L]

    def aux_loss(self, T=None, fbar_prev=None, replicas=1):
        """``replicas``: the statistics were summed over this many data-parallel replicas of T tokens."""
        T = (self.T if T is None else T) * replicas
        c = self.ctx
        if fbar_prev is not None and fbar_prev.dim() == 1:
            fbar_prev = fbar_prev.reshape(1, -1)
        for g in range(self.G):
            l0 = g * self.Lg
            c.pool_aux_loss(self.counts[l0:l0 + self.Lg], self.score_sum[l0:l0 + self.Lg], self.Lg, self.m, T,
                            self.alpha, None if fbar_prev is None else fbar_prev[g],
                            self.loss[g:g + 1], self.coef[g], self.fbar[g])
        return self.loss

    # ------------------------------------------------------------------ backward
    def backward_layer(self, l, dx_next, dx_out, T=None, with_aux=True, overwrite=False):
        """``overwrite``: this layer's weight gradient replaces what the pool-gradient
        slices of its view hold (the first contribution of a step) instead of adding to it."""
        T = self.T if T is None else T
        c = self.ctx
        s = l if self.deferred_wgrad else 0
        a = self.slot(l)
        if self.recompute:
            self.permute_and_experts(l, T)
        flags = B.BWD_SKIP_WGRAD if self.deferred_wgrad else (B.WGRAD_OVERWRITE if overwrite else 0)
        c.expert_bwd(dx_next, T, self.row_of[l], self.gate[l], self.token_of[l], self.offsets[l],
                     self.tile_expert[l], self.Xp[a], self.GU[a], self.A[a], self.Yp[a], self.W_gu,
                     self.W_down, self.base(l), self.m, dx_next, self.dYp[s], self.dGU[s], dx_out,
                     self.dgate, self.dW_gu, self.dW_down, flags)
        coef = None
        if with_aux:
            coef = self.coef[l // self.Lg]
        c.route_bwd(self.x[l], T, self.W_r[l], self.sigma[l], self.m, self.znorm[l], self.z[l],
                    self.idx[l], self.dgate, coef, dx_out, self.dW_r[l], self.dsigma[l:l + 1])

    def backward(self, upstream=None, T=None, with_aux=True, accumulate=True, exchange=None):
        """``accumulate=False``: the pool gradient of this pass replaces the buffers' contents
        (the first weight-gradient contribution to each expert is a store, the rest add), so the
        buffers need no zeroing; router gradients always add.  ``exchange`` (a
        ``dp.GradientExchange``): the gradients are summed over the data-parallel replicas, each
        buffer as soon as it is complete (dW_down while dW_gu is still being computed)."""
        T = self.T if T is None else T
        cur = 0
        if upstream is not None:
            self.dx[cur, :T].copy_(upstream, non_blocking=True)
        for l in reversed(range(self.L)):
            first = (not accumulate) and l % self.Lg == self.Lg - 1     # first contribution to its group's experts
            self.backward_layer(l, self.dx[cur], self.dx[1 - cur], T, with_aux, overwrite=first)
            cur = 1 - cur
        if self.deferred_wgrad:
            for g in range(self.G):                        # one pass per sharing group over its layers
                l0 = g * self.Lg
                flags = 0 if accumulate else B.WGRAD_OVERWRITE
                args = (self.Lg, self.cap, self.offsets[l0:], self.Xp[l0:], self.A[l0:], self.dYp[l0:],
                        self.dGU[l0:], g * self.m, self.m)
                if exchange is None:
                    self.ctx.pool_wgrad(*args, self.dW_gu, self.dW_down, flags)
                else:
                    e0, e1 = g * self.m, (g + 1) * self.m
                    self.ctx.pool_wgrad(*args, None, self.dW_down, flags)
                    exchange.launch([self.dW_down[e0:e1]])
                    self.ctx.pool_wgrad(*args, self.dW_gu, None, flags)
                    exchange.launch([self.dW_gu[e0:e1]])
        if exchange is not None:
            if not self.deferred_wgrad:
                exchange.launch([self.dW_down, self.dW_gu])
            exchange.launch([self.dW_r, self.dsigma])
            exchange.finish()
        return self.dx[cur]

    def step(self, x0=None, upstream=None, T=None, accumulate=True, exchange=None, out=None):
        """One pass of the whole hot path: forward, balance loss, backward.  With ``exchange`` the
        step is one data-parallel replica's: the balance loss is taken on the statistics of all
        replicas' tokens and the gradients are summed over the replicas.
        Host-resident tensors (pinned memory) are moved beside the compute on a second stream: an
        ``upstream`` on the host is copied in while the forward pass runs, and ``out`` (host or
        device, [T, d]) receives x_L while the backward pass runs; both copies are ordered before
        the step's end on the calling stream."""
        T_ = self.T if T is None else T
        cur = torch.cuda.current_stream(self.device)
        side = None
        up_ready = None
        if (upstream is not None and not upstream.is_cuda) or out is not None:
            if self._copy_stream is None:
                self._copy_stream = torch.cuda.Stream(self.device)
            side = self._copy_stream
            side.wait_stream(cur)                          # nothing queued before this step still uses dx / out
        if upstream is not None and not upstream.is_cuda:
            with torch.cuda.stream(side):
                self.dx[0, :T_].copy_(upstream, non_blocking=True)
                up_ready = side.record_event()
            upstream = None                                # backward starts from dx[0]
        self.forward(x0, T)
        if out is not None:
            side.wait_stream(cur)
            with torch.cuda.stream(side):
                out.copy_(self.x[self.L, :T_], non_blocking=True)
        replicas = 1 if exchange is None else exchange.global_statistics(self.counts, self.score_sum)
        self.aux_loss(T, replicas=replicas)
        if not accumulate:
            self.zero_router_grad()
        if up_ready is not None:
            cur.wait_event(up_ready)
        dx0 = self.backward(upstream, T, accumulate=accumulate, exchange=exchange)
        if side is not None:
            cur.wait_stream(side)
        return dx0

    def accumulate_microbatches(self, batches, fbar0=None, T=None, exchange=None):
        """One optimizer step's worth of the path (App. D, App. G): every micro-batch (x0, upstream)
        runs forward, balance loss and backward; all of them add into the same gradient buffers (the
        first one overwrites them), and the balance loss of a micro-batch uses the token fractions
        f-bar of the PREVIOUS micro-batch - ``fbar0`` for the first (default: the f-bar this stack saw
        last, or uniform 1/m).  Returns the per-micro-batch losses (device tensors).
        With ``exchange`` (data-parallel replicas): f-bar of a micro-batch is summed over the
        replicas (each replica's part is its counts over the whole batch's assignments) while its
        backward pass runs - the lagged scheme needs no statistic of the current micro-batch, so no
        reduction sits between forward and backward -, each loss returned is this
        replica's share of the whole batch's (they add up over the replicas), and the gradients are
        summed over the replicas once, after the last micro-batch."""
        if fbar0 is not None:
            self.fbar_lag = fbar0.to(self.device, torch.float32).reshape(self.fbar.shape).clone()
        elif self.fbar_lag is None:
            self.fbar_lag = torch.full_like(self.fbar, 1.0 / self.m)
        losses = []
        self.zero_router_grad()
        replicas = 1 if exchange is None else exchange.world
        n = len(batches)
        for i, (x0, upstream) in enumerate(batches):
            self.forward(x0, T)
            if exchange is not None:
                exchange.finish()                      # the previous micro-batch's f-bar has arrived
            self.aux_loss(T, fbar_prev=self.fbar_lag, replicas=replicas)
            losses.append(self.loss.clone())
            self.fbar_lag.copy_(self.fbar)             # updated after all layers finished forward, no gradient
            if exchange is not None:
                exchange.launch([self.fbar_lag])
            self.backward(upstream, T, accumulate=i > 0, exchange=exchange if i == n - 1 else None)
        return losses

    def capture_step(self, x0=None, upstream=None, accumulate=True, out=None):
        """Records one whole step (the library calls of ``step`` with these tensors) into a CUDA graph
        and returns it; ``graph.replay()`` then issues the step with one launch.  Every call of the
        path is asynchronous on the stream and allocates nothing, so the recording holds exactly the
        kernels and copies an eager step issues."""
        side = torch.cuda.Stream(self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(side):                       # one eager pass first: lazy set-up happens here
            self.step(x0, upstream, accumulate=accumulate, out=out)
        torch.cuda.current_stream(self.device).wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            self.step(x0, upstream, accumulate=accumulate, out=out)
        return graph

    def close(self):
        self.ctx.close()
