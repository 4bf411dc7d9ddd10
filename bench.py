#!/usr/bin/env python
"""Benchmark of the UniPool MoE-layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one pass of the whole hot path over one synthetic batch: for every
layer route -> dispatch -> grouped expert FFN -> combine, then the pool balance
loss, then for every layer (in reverse) expert backward (dgrad + wgrad into the
shared fp32 pool gradient) and router backward.  The metric is MoE-layer
fwd+bwd tokens per second: tokens * layers / step time, summed over all GPUs
(each rank runs the same workload on its own token shard; no data-path
collective - the layer is token-parallel).

Prints ONE JSON line (rank 0).  The line's headline numbers are those of `--workload` (default: the
978M-shaped stack, the largest configuration that fits one GPU); at N = 1 a compact `workloads`
block adds the 182M-shaped stack, its layer-private ("vanilla") layout, the reduced pool and the
skewed fine-grained stack, each timed the same way.  `--gpus N` without a launcher's environment
starts the N ranks itself (torch.distributed.run, one process per GPU); with N > 1 the line carries
both the independent-replica step and the data-parallel step whose statistics and gradients are
summed over the ranks.  `--impl reference` times the CPU oracle, as it stands, on a bounded sample
of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of a workload's dominant kernel,
# from the ncu capture summarised in profiles/grouped_gemm_978m_slice_ncu.txt: the 978m_slice case (an
# eighth of the experts and of the rows of one 978m layer) moved 733.9 + 207.8 MB; a full launch is eight
# times that (weights and activations both grow with the units processed).
NCU_TRAFFIC = {("978m", "expert_fwd_gu"): 8 * (733.89e6 + 207.79e6)}

# kernel behind each grouped-GEMM phase (for the roofline's `kernel` field) and launches of one dispatch-map call
GEMM_KERNEL = {"expert_fwd_gu": "grouped_gemm_tc_kernel", "expert_fwd_down": "grouped_gemm_tc_kernel",
               "dgrad_down": "grouped_gemm_tc_kernel", "dgrad_gu": "grouped_gemm_tc_kernel",
               "wgrad_down": "wgrad_pair_kernel", "wgrad_gu": "wgrad_pair_kernel"}
DISPATCH_MAP_LAUNCHES = 1

METRIC = "moe_layer_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"

# algorithmic FLOPs of the grouped GEMM phases per routed row: 2*d*f per (row, GEMM of d x f)
GEMM_PHASES = {"expert_fwd_gu": 4, "expert_fwd_down": 2, "dgrad_down": 2, "dgrad_gu": 4, "wgrad_down": 2,
               "wgrad_gu": 4}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi every 50 ms; the summary covers the
    samples that arrived between ``begin()`` and ``end()`` (the timed region)."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.t_begin = self.t_end = None

    def begin(self):
        self.t_begin = time.perf_counter()

    def end(self):
        self.t_end = time.perf_counter()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [l for t, l in self.lines if self.t_begin is not None and self.t_begin <= t <= self.t_end]
        for line in inside or [l for _, l in self.lines]:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return dict(sm_mhz=sm[len(sm) // 2] if sm else None, sm_max_mhz=max(smax) if smax else None,
                    power_w_max=max(power) if power else None, samples=len(sm),
                    window="timed region" if inside else "whole run", reasons=sorted(reasons))


def algorithmic_bytes(cfg, cap_rows):
    """HBM bytes the memory-bound phases must move per launch (bf16 activations)."""
    T, d, k, m = cfg["T"], cfg["d"], cfg["k"], (cfg["private"] or cfg["M"])
    R = T * k
    b = 2
    if cfg["dtype"] == "bf16":
        # tensor-core router: "route_logits" is the split of W_r into bf16 terms (a few hundred KB, no
        # bandwidth figure), "route_select" the fused kernel that reads x, writes the logits and does
        # scoring, top-k and statistics
        route = {"route_select": T * d * b + T * m * 4 + T * k * 8 + T * 4 + 3 * m * d * 2}
    else:
        route = {"route_logits": T * d * 4 + T * m * 4 + m * d * 4, "route_select": T * m * 4 + T * k * 8 + T * 4}
    return {
        **route,
        "dispatch_gather": T * d * b + R * d * b + R * 4,
        "combine": R * d * b + 2 * T * d * b + T * k * 8,
        "bwd_scale_gather": T * d * b + 2 * R * d * b + T * k * 12,     # dy + Yp read, dYp written, dgate
        "unpermute_sum": R * d * b + 2 * T * d * b + T * k * 4,
    }


def measure_workload(name, args, world, rank, dev, full):
    """Times one workload on this rank's GPU and returns its figures.  ``full``: the headline
    workload (clock samples, end-to-end leg, per-kernel table); otherwise a compact summary."""
    import torch
    import torch.distributed as dist
    from paper_2605_06665_b200 import binding as B
    from paper_2605_06665_b200 import dp, synth
    from paper_2605_06665_b200.stack import UniPoolStack

    cfg = dict(synth.CONFIGS[name])
    L, T, d, f, M, k = cfg["L"], cfg["T"], cfg["d"], cfg["f"], cfg["M"], cfg["k"]
    m = synth.router_width(cfg)
    steps = args.steps if full else max(3, min(args.steps, 5))
    inputs = synth.make_inputs(cfg, seed=dp.shard_seed(rank))
    small = B.Context(B.make_config(64, 64, m, k, 1, 128, B.FP32, synth.EPS, 1.0), dev)
    c_val = small.calibrate_c(m, k, 100_000, seed=0)           # Alg. 1 on the device
    small.close()
    del small
    st = UniPoolStack(L, d, f, M, k, T, cfg["dtype"], cfg["private"], c=c_val, eps=synth.EPS, alpha=synth.ALPHA,
                      device=dev, deferred_wgrad=args.deferred_wgrad, router=cfg.get("router", "norm"))
    st.load(inputs["pool"], inputs["routers"])
    tdt = st.tdtype
    x0_host = torch.from_numpy(inputs["x0"]).to(tdt).pin_memory()
    up_host = torch.from_numpy(inputs["upstream"]).to(tdt).pin_memory()
    del inputs
    x0 = x0_host.to(dev)
    up = up_host.to(dev)
    xL_host = torch.empty_like(x0_host).pin_memory()
    loss_host = torch.empty(st.loss.shape, dtype=torch.float32).pin_memory()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, n):
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        sync_all()
        return dp.max_over_ranks(e0.elapsed_time(e1), world, dev)

    def device_step():
        # the step's first weight-gradient contribution overwrites the fp32 pool gradient, so it
        # needs no zeroing; the (small) router gradients are zeroed inside the step
        st.step(x0, up, accumulate=False)

    def e2e_step():
        # H2D copies of this step's inputs from pinned memory, D2H of x_L (beside the compute) and of the loss
        st.step(x0_host, up_host, accumulate=False, out=xL_host)
        loss_host.copy_(st.loss, non_blocking=True)

    eager_step = device_step
    if args.graph:                           # one CUDA graph per step variant: same kernels, one launch
        g_dev = st.capture_step(x0, up, accumulate=False)
        device_step = g_dev.replay
        if full:
            g_e2e = st.capture_step(x0_host, up_host, accumulate=False, out=xL_host)

            def e2e_step():
                g_e2e.replay()
                loss_host.copy_(st.loss, non_blocking=True)
    sampler = ClockSampler(dev.index)                # started ahead of the warm-up: the first sample takes a while
    if rank == 0 and full and not args.kernels_only:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        device_step()
    st.ctx.check_status()
    if args.kernels_only:                    # profiler runs: nothing but the steps themselves
        timed(device_step, steps)
        st.ctx.check_status()
        st.close()
        return {"kernels_only": True, "workload": name, "steps": steps}
    sampler.begin()
    ms_total = timed(device_step, steps)
    sampler.end()
    clocks = sampler.stop() if rank == 0 and full else None

    # per-kernel durations, measured live with CUDA events on the launch stream
    st.ctx.profile_enable(True)
    timed(eager_step, steps)
    prof = st.ctx.profile_read()
    st.ctx.profile_enable(False)

    ms_e2e = None
    if full:
        for _ in range(2):
            e2e_step()
        ms_e2e = timed(e2e_step, steps)

    # the data-parallel step (N > 1): routing statistics summed over the ranks before the balance
    # loss, gradients summed as they complete (the pool's dW_down travels while dW_gu is computed);
    # issued eagerly - the collectives are not part of a recorded graph
    ms_exchange = None
    if full and (world > 1 or args.grad_exchange):
        exchange = dp.GradientExchange(world)

        def exchange_step():
            st.step(x0, up, accumulate=False, exchange=exchange)

        for _ in range(2):
            exchange_step()
        ms_exchange = timed(exchange_step, steps)
    st.ctx.check_status()

    ms_step = ms_total / steps
    peaks = _peaks()
    R = T * k
    kernels = {}
    for kname, (ms, launches) in prof.items():
        if launches == 0:
            continue
        calls = launches / max(1, DISPATCH_MAP_LAUNCHES if kname == "dispatch_maps" else 1)
        kernels[kname] = dict(ms_per_step=ms / steps, launches_per_step=launches // steps, ms_per_call=ms / calls)
    abytes = algorithmic_bytes(cfg, st.cap)
    for kname, factor in GEMM_PHASES.items():
        if kname in kernels:
            flops = factor * R * d * f * L               # per step, whatever the number of launches
            tf = flops / (kernels[kname]["ms_per_step"] * 1e-3) / 1e12
            kernels[kname].update(tflops=tf, frac_of_measured_sustained=tf / peaks["bf16_tflops_sustained"])
    for kname, nbytes in abytes.items():
        if kname in kernels:
            gbs = nbytes / (kernels[kname]["ms_per_call"] * 1e-3) / 1e9
            kernels[kname].update(gbs=gbs, frac_of_measured_hbm=gbs / peaks["hbm_gbs"])
    # every grouped GEMM also has an HBM floor: the pool weights its experts own are read once per
    # launch, activations once; the bound of a phase is the larger of its two floors
    mw = (cfg["private"] or M)                           # experts whose weights one layer's launch reads
    wbytes = {"expert_fwd_gu": 2 * f * d, "expert_fwd_down": d * f, "dgrad_down": d * f, "dgrad_gu": 2 * f * d}
    abytes_gemm = {"expert_fwd_gu": R * (d + 3 * f), "expert_fwd_down": R * (f + d), "dgrad_down": R * (d + 4 * f),
                   "dgrad_gu": R * (2 * f + d), "wgrad_down": R * (d + f), "wgrad_gu": R * (2 * f + d)}
    wgrad_once = bool(st.deferred_wgrad) or bool(cfg["private"])   # the fp32 gradient is written exactly once
    for kname in GEMM_PHASES:
        if kname not in kernels:
            continue
        nbytes = L * 2 * abytes_gemm[kname]
        if kname in wbytes:
            nbytes += L * mw * wbytes[kname] * 2
        else:
            per_pool = M * (d * f if kname == "wgrad_down" else 2 * f * d) * 4
            nbytes += per_pool if wgrad_once else per_pool * (2 * L - 1)
        t = kernels[kname]["ms_per_step"] * 1e-3
        t_tensor = GEMM_PHASES[kname] * R * d * f * L / (peaks["bf16_tflops_sustained"] * 1e12)
        t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
        kernels[kname].update(hbm_bytes_per_step=nbytes, gbs=nbytes / t / 1e9,
                              frac_of_measured_hbm=nbytes / t / 1e9 / peaks["hbm_gbs"],
                              bound="hbm" if t_hbm > t_tensor else "tensor",
                              frac_of_ceiling=max(t_hbm, t_tensor) / t)
    gemm_ms = {n: kernels[n]["ms_per_step"] for n in GEMM_PHASES if n in kernels}
    dominant = max(gemm_ms, key=gemm_ms.get)
    dom = kernels[dominant]
    # the library runs the row-tile GEMMs on CTA pairs when a full batch gives the average expert of a
    # layer's view four row tiles of 128 rows
    kernel_name = GEMM_KERNEL[dominant]
    if kernel_name == "grouped_gemm_tc_kernel" and T * k >= 4 * 128 * mw:
        kernel_name = "row_pair_kernel"
    # per launch of the dominant kernel: algorithmic bytes / FLOPs over its average CUDA-event duration
    if dom["bound"] == "hbm":
        roofline = dict(kernel=kernel_name + ":" + dominant, bound="hbm", achieved=dom["gbs"],
                        peak=peaks["hbm_gbs"], unit="GB/s", frac=dom["gbs"] / peaks["hbm_gbs"],
                        peak_source=peaks["source"], traffic=None,
                        tensor_tflops=dom["tflops"], tensor_frac_of_sustained=dom["frac_of_measured_sustained"])
    else:
        roofline = dict(kernel=kernel_name + ":" + dominant, bound="tensor", achieved=dom["tflops"],
                        peak=peaks["bf16_tflops_sustained"], unit="TFLOP/s",
                        frac=dom["tflops"] / peaks["bf16_tflops_sustained"],
                        peak_source=peaks["source"] + " sustained", traffic=None, hbm_gbs=dom["gbs"])
    roofline["traffic"] = NCU_TRAFFIC.get((name, dominant))
    ceiling_s = sum(kernels[n]["ms_per_step"] * 1e-3 * kernels[n]["frac_of_ceiling"] for n in gemm_ms)
    total_gemm_flops = 18 * R * d * f * L
    gemm_time = sum(gemm_ms.values()) * 1e-3
    launches = sum(v["launches_per_step"] for v in kernels.values())
    non_gemm_ms = sum(v["ms_per_step"] for n, v in kernels.items() if n not in GEMM_PHASES)
    summary = {
        "ms_per_step": ms_step, "value": dp.whole_job_throughput(T * L, world, ms_step), "steps": steps,
        "gemm_tflops_all_phases": total_gemm_flops / gemm_time / 1e12,
        "gemm_frac_of_measured_sustained": total_gemm_flops / gemm_time / 1e12 / peaks["bf16_tflops_sustained"],
        "gemm_frac_of_ceiling": ceiling_s / gemm_time,      # sum of per-phase max(tensor, HBM) floors / measured
        "non_gemm_ms_per_step": non_gemm_ms,
        "roofline": roofline,
    }
    if not full:
        summary["phases"] = {n: {q: v[q] for q in ("ms_per_step", "tflops", "gbs", "bound", "frac_of_ceiling",
                                                    "frac_of_measured_hbm") if q in v}
                             for n, v in kernels.items()}
        st.close()
        return summary
    out = {
        "metric": METRIC, "value": summary["value"], "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg["dtype"], "data": "synthetic",
        "config": {"workload": name, "layers": L, "d_model": d, "d_ff": f, "pool_experts": M, "top_k": k,
                   "tokens_per_gpu": T, "layout": "private" if cfg["private"] else "shared_pool",
                   "deferred_wgrad": bool(st.deferred_wgrad), "cuda_graph": bool(args.graph),
                   "l2": "working set per step (weights + saved activations, several GB) exceeds the 126 MB L2",
                   "norm_router_c": c_val},
        "clocks": clocks,
        "e2e": {"value": dp.whole_job_throughput(T * L, world, ms_e2e / steps), "unit": UNIT,
                "ms_per_step": ms_e2e / steps,
                "h2d_bytes_per_step": int(x0_host.numel() * x0_host.element_size() * 2),
                "d2h_bytes_per_step": int(xL_host.numel() * xL_host.element_size() + loss_host.numel() * 4)},
        "gpu_launches": launches * steps,
        "roofline": roofline,
        "stack_tokens_per_s": world * T / (ms_step * 1e-3),
        "gemm_tflops_all_phases": summary["gemm_tflops_all_phases"],
        "gemm_frac_of_measured_sustained": summary["gemm_frac_of_measured_sustained"],
        "gemm_frac_of_ceiling": summary["gemm_frac_of_ceiling"],
        "non_gemm_ms_per_step": non_gemm_ms,
        "kernels": kernels,
    }
    if ms_exchange is not None:
        # the same step with the one exchange of data-parallel training inside it (App. D)
        out["grad_exchange"] = {"ms_per_step": ms_exchange / steps,
                                "value": dp.whole_job_throughput(T * L, world, ms_exchange / steps), "unit": UNIT,
                                "allreduce_bytes_per_step": int(4 * (st.dW_gu.numel() + st.dW_down.numel() +
                                                                     st.dW_r.numel() + st.dsigma.numel())),
                                "cuda_graph": False}
    st.close()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    from paper_2605_06665_b200 import dp

    world, rank, local_rank = dp.env_world()
    if rank == 0:
        entry.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    if rank != 0:
        from paper_2605_06665_b200 import binding
        binding.lib()
    dev = torch.device("cuda", local_rank)

    out = measure_workload(args.workload, args, world, rank, dev, full=True)
    torch.cuda.empty_cache()
    if not args.kernels_only and world == 1:
        from paper_2605_06665_b200 import synth
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(dict(synth.CONFIGS[args.workload]), budget_tokens=args.cpu_tokens)
        extra = [w for w in args.extra_workloads.split(",") if w and w != args.workload]
        block = {}
        for w in extra:
            block[w] = measure_workload(w, args, world, rank, dev, full=False)
            torch.cuda.empty_cache()
        if block:
            out["workloads"] = block
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] or [1]))
    except Exception:
        return len(os.sched_getaffinity(0))


def oracle_layer_step(cfg, inputs, Ts):
    """One MoE layer (forward, balance-loss term, backward with all gradients) of the CPU oracle, as it
    stands, over the first Ts tokens of `inputs`; float32 arithmetic (the arrays it is fed are float32).
    Returns the seconds it took."""
    import numpy as np
    from oracle import unipool_oracle as O
    from paper_2605_06665_b200 import synth
    pool, router = inputs["pool"], dict(inputs["routers"][0], mode=cfg.get("router", "norm"))
    k = cfg["k"]
    t0 = time.perf_counter()
    cache = O.layer_forward(inputs["x0"][:Ts], router, pool, k, np.float32(2.0), np.float32(synth.EPS))
    _, _, coef = O.pool_aux_loss(cache["counts"][None], cache["S"][None], Ts, k, synth.ALPHA)
    grad = O.zeros_like_pool(pool)
    O.layer_backward(cache, router, pool, k, np.float32(2.0), np.float32(synth.EPS), inputs["upstream"][:Ts],
                     coef.astype(np.float32), grad)
    return time.perf_counter() - t0


def oracle_sample_text(cfg, Ts):
    return (f"one MoE layer fwd+bwd (route, Eq. 2, balance-loss term, all gradients) over {Ts} of the "
            f"{cfg['T']} tokens, full pool of {cfg['M']} experts, float32 numpy")


def cpu_baseline(cfg, budget_tokens=2048):
    """Times the CPU oracle on one MoE layer over a token sample of the workload."""
    from paper_2605_06665_b200 import synth
    Ts = min(budget_tokens, cfg["T"])
    inputs = synth.make_inputs(cfg, seed=0, T=Ts, L=1)
    sec = oracle_layer_step(cfg, inputs, Ts)
    return dict(value=Ts / sec, unit=UNIT, cores=oracle_threads(), kind="oracle", seconds=sec,
                sample=oracle_sample_text(cfg, Ts))


def run_reference(args):
    """The reference arm is the oracle (the paper ships no implementation): W warm-up steps, then exactly K
    timed steps, each one layer over the same token sample; the sample is halved until the projected run
    fits the time budget."""
    from paper_2605_06665_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__ as entry  # noqa: F401  (path set-up)
    cfg = dict(synth.CONFIGS[args.workload])
    Ts = min(args.ref_tokens, cfg["T"])
    inputs = synth.make_inputs(cfg, seed=0, T=Ts, L=1)
    n_total = args.steps + max(args.warmup, 1)
    first = oracle_layer_step(cfg, inputs, Ts)                      # warm-up step 1, also the probe
    while first * n_total > args.ref_budget_s and Ts > 256:
        Ts //= 2
        first = oracle_layer_step(cfg, inputs, Ts)
    for _ in range(args.warmup - 1):
        oracle_layer_step(cfg, inputs, Ts)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_layer_step(cfg, inputs, Ts)
    sec = (time.perf_counter() - t0) / max(args.steps, 1)
    value = Ts / sec
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "note": "CPU oracle; each step = one MoE layer fwd+bwd over a token sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": oracle_sample_text(cfg, Ts)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="978m")
    ap.add_argument("--extra-workloads", default="182m,182m_vanilla,182m_pool40,fine_zipf",
                    help="comma-separated workloads summarised in the line's `workloads` block (N = 1 only; "
                         "'' for none)")
    ap.add_argument("--per-layer-wgrad", dest="deferred_wgrad", action="store_false",
                    help="accumulate each layer's weight gradient into the pool gradient during that layer's "
                         "backward instead of contracting all layers' rows per expert in one pass at the end")
    ap.add_argument("--cpu-tokens", type=int, default=16384, help="token sample of the CPU-oracle baseline")
    ap.add_argument("--ref-tokens", type=int, default=4096,
                    help="--impl reference: tokens per step of the oracle (halved while the run would exceed the budget)")
    ap.add_argument("--ref-budget-s", type=float, default=240.0, help="--impl reference: time budget of the whole run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--grad-exchange", action="store_true",
                    help="also time the data-parallel step (routing statistics and gradients summed over the "
                         "ranks inside the step) at N = 1; with N > 1 it is always timed beside the replica step")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="issue every library call of a step eagerly instead of replaying one CUDA graph")
    ap.add_argument("--kernels-only", action="store_true",
                    help="run warm-up and timed steps only and print no result (for runs under a profiler)")
    args = ap.parse_args()
    from paper_2605_06665_b200 import dp
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher above us: start the N ranks ourselves, one process per GPU
        sys.exit(dp.launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
