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


def test_single_rank_is_the_identity():
    from paper_2605_06665_b200 import dp
    assert dp.max_over_ranks(3.5, 1) == 3.5
    assert dp.whole_job_throughput(100, 1, 10.0) == 1e4
