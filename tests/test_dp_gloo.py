"""The benchmark's multi-rank plumbing on CPU: two gloo ranks, each with its own token shard; the
reported time is the slowest rank's and the throughput counts every rank's tokens."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_2605_06665_b200 import dp, synth
    world, rank, local = dp.env_world()
    dist.init_process_group("gloo")
    cfg = dict(synth.CONFIGS["tiny_fp32"])
    x = synth.make_inputs(cfg, seed=dp.shard_seed(rank), T=8, L=1)["x0"]
    dist.barrier()
    ms = dp.max_over_ranks(10.0 + 5.0 * rank, world)           # rank 1 is the slow one
    out = dict(rank=rank, world=world, ms=ms, value=dp.whole_job_throughput(8 * 1, world, ms),
               first=float(x[0, 0]))
    print("RESULT " + json.dumps(out), flush=True)
    dist.barrier()
    dist.destroy_process_group()
""" % ROOT)


def test_two_gloo_ranks_report_the_slowest_time_and_all_tokens(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    results = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        results.append(json.loads([l for l in out.splitlines() if l.startswith("RESULT ")][0][7:]))
    assert sorted(r["rank"] for r in results) == [0, 1]
    for r in results:
        assert r["world"] == 2 and r["ms"] == 15.0                      # the slowest rank's time, on every rank
        assert abs(r["value"] - 2 * 8 / 15e-3) < 1e-6                   # both ranks' tokens
    assert results[0]["first"] != results[1]["first"]                   # different token shards


EXCHANGE_WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch
    import torch.distributed as dist
    from paper_2605_06665_b200 import dp
    from oracle import unipool_oracle as O
    world, rank, local = dp.env_world()
    dist.init_process_group("gloo")
    ex = dp.GradientExchange(world)
    rng = np.random.default_rng(7)                       # every rank draws the same whole batch
    L, M, d, f, k, T = 3, 6, 8, 5, 2, 12
    pool = dict(W_gate=rng.normal(0, .5, (M, f, d)), W_up=rng.normal(0, .5, (M, f, d)), W_down=rng.normal(0, .5, (M, d, f)))
    routers = [dict(W_r=rng.normal(0, .5, (M, d)), sigma=1.0 + .1 * l, bias=None) for l in range(L)]
    x0, up = rng.normal(0, 1, (T, d)), rng.normal(0, 1, (T, d))
    whole = O.stack_objective_and_grads(x0, routers, pool, k, 1.7, 1e-6, 0.3, up)
    mine = slice(rank * T // world, (rank + 1) * T // world)

    def summed(counts, S):                               # the statistics exchange of the replica step
        cn, ss = torch.from_numpy(counts.astype(np.int32)), torch.from_numpy(S.astype(np.float32))
        n = ex.global_statistics(cn, ss)
        return cn.numpy().astype(np.int64), ss.numpy().astype(np.float64), n * (T // world)

    res = O.stack_objective_and_grads(x0[mine], routers, pool, k, 1.7, 1e-6, 0.3, up[mine], replica_stats=summed)
    grads = [torch.from_numpy(np.ascontiguousarray(res["pool_grad"][n], dtype=np.float32)) for n in ("W_down", "W_gate", "W_up")]
    dW_r = torch.from_numpy(np.stack([g["dW_r"] for g in res["router_grads"]]).astype(np.float32))
    ex.launch(grads[:1])                                 # dW_down leaves first ...
    ex.launch(grads[1:] + [dW_r])                        # ... the rest while it travels
    ex.finish()
    err = max(float(np.abs(g.numpy() - whole["pool_grad"][n]).max() / np.abs(whole["pool_grad"][n]).max())
              for g, n in zip(grads, ("W_down", "W_gate", "W_up")))
    ref_r = np.stack([g["dW_r"] for g in whole["router_grads"]])
    err_r = float(np.abs(dW_r.numpy() - ref_r).max() / np.abs(ref_r).max())
    out = dict(rank=rank, err=err, err_r=err_r, loss=float(res["loss_aux"]), whole_loss=float(whole["loss_aux"]),
               pending=len(ex._pending))
    print("RESULT " + json.dumps(out), flush=True)
    dist.barrier()
    dist.destroy_process_group()
""" % ROOT)


def _run_two_ranks(tmp_path, source):
    import json
    script = tmp_path / "worker.py"
    script.write_text(source)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    results = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        results.append(json.loads([l for l in out.splitlines() if l.startswith("RESULT ")][0][7:]))
    return results


def test_two_replicas_exchange_statistics_and_gradients(tmp_path):
    """Two gloo replicas, half of the batch each: after the statistics and gradient exchange every
    replica holds the whole batch's balance loss and the whole batch's gradients (the oracle computes
    both sides; the exchange itself is the library's)."""
    results = _run_two_ranks(tmp_path, EXCHANGE_WORKER)
    assert sorted(r["rank"] for r in results) == [0, 1]
    for r in results:
        assert r["err"] < 1e-6 and r["err_r"] < 1e-6          # float32 transport of float64 gradients
        assert abs(r["loss"] - r["whole_loss"]) <= 1e-6 * abs(r["whole_loss"])
        assert r["pending"] == 0


def test_single_rank_is_the_identity():
    import torch
    from paper_2605_06665_b200 import dp
    ex = dp.GradientExchange(1)
    t = torch.arange(4.0)
    assert ex.global_statistics(torch.ones(3, dtype=torch.int32), torch.ones(3)) == 1
    ex.launch([t])
    ex.finish()
    assert t.tolist() == [0.0, 1.0, 2.0, 3.0]
    assert dp.max_over_ranks(3.5, 1) == 3.5
    assert dp.whole_job_throughput(100, 1, 10.0) == 1e4


LAUNCHED = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_2605_06665_b200 import dp
    world, rank, local = dp.env_world()
    dist.init_process_group("gloo")
    ms = dp.max_over_ranks(1.0 + rank, world)
    with open(os.path.join(sys.argv[1], "rank%%d.json" %% rank), "w") as fh:
        json.dump(dict(world=world, rank=rank, local=local, ms=ms, argv=sys.argv[2:]), fh)
    dist.barrier()
    dist.destroy_process_group()
""" % ROOT)


def test_launcher_starts_one_process_per_rank(tmp_path):
    """`bench.py --gpus N` without a launcher's environment starts its ranks through dp.launch_ranks:
    here a stub worker stands in for the benchmark (gloo, CPU)."""
    import json
    sys.path.insert(0, ROOT)
    from paper_2605_06665_b200 import dp
    script = tmp_path / "stub.py"
    script.write_text(LAUNCHED)
    cmd = dp.launch_command(2, str(script), ["x"], 12345)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-2:] == [str(script), "x"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    rc = dp.launch_ranks(2, str(script), [str(tmp_path), "--steps", "3"], env=env)
    assert rc == 0
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    for r, g in enumerate(got):
        assert g["world"] == 2 and g["rank"] == r and g["local"] == r
        assert g["ms"] == 2.0 and g["argv"] == ["--steps", "3"]
