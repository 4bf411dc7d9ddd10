"""Data-parallel plumbing of the benchmark: the MoE-layer path shards over tokens with no
collective inside the layer (each rank holds the pool and all routers and runs the whole path on its
own token shard), so the only cross-rank steps are the barrier around the timed region and the
max-over-ranks of the measured time.  ``torch.distributed`` does both (NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

import os


def env_world():
    """(world_size, rank, local_rank) from the launcher's environment (1, 0, 0 when absent)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def free_port():
    """A TCP port that is free on 127.0.0.1 right now (for the ranks' rendezvous)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def launch_command(n_ranks, script, argv, port):
    """The command that runs ``script argv`` as ``n_ranks`` processes of one node (one per GPU) under
    ``torch.distributed.run``; the ranks meet on 127.0.0.1:``port``."""
    import sys
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n_ranks)}",
            "--master-addr", "127.0.0.1", "--master-port", str(int(port)), script] + list(argv)


def launch_ranks(n_ranks, script, argv, env=None):
    """Starts the ranks (see ``launch_command``), waits for them and returns the launcher's exit code.
    The children find RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in their environment."""
    import subprocess
    return subprocess.call(launch_command(n_ranks, script, argv, free_port()), env=env)


def shard_seed(rank):
    """Seed of rank ``rank``'s synthetic token shard: every rank draws its own tokens."""
    return int(rank)


def max_over_ranks(value, world, device="cpu"):
    """Largest ``value`` (a float, e.g. elapsed milliseconds) over all ranks; the identity when world == 1."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank, world, ms):
    """Units all ranks processed per second, given the slowest rank's time in milliseconds (weak scaling)."""
    return world * units_per_rank / (ms * 1e-3)


class GradientExchange:
    """The one exchange of a data-parallel training step around the MoE path (the paper's own
    parallel mode, App. D: data parallel, no expert parallelism): every replica holds the pool and
    all routers, runs the whole path on its token shard, and the replicas then sum

      * the routing statistics ``counts, score_sum [L, m]`` (before the balance loss, so that the
        token fractions and mean scores of Eqs. 3-5 are those of the whole batch), and
      * the fp32 gradients of the pool, the routers and the router scales.

    Reductions are issued asynchronously (``launch``): the collective waits for the work queued so
    far on the current stream and runs beside what is queued after it, so the pool's dW_down can
    travel while dW_gu is still being computed; ``finish`` makes the current stream (NCCL) or the
    host (gloo) wait for all of them.  With one replica every method is the identity.
    """

    def __init__(self, world, group=None):
        self.world = int(world)
        self.group = group
        self._pending = []

    def global_statistics(self, counts, score_sum):
        """Sums ``counts`` (int32) and ``score_sum`` (float32) over the replicas in place and returns
        the factor by which the token count of the balance loss grows (the number of replicas: every
        replica runs the same number of tokens)."""
        if self.world > 1:
            import torch.distributed as dist
            dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=self.group)
            dist.all_reduce(score_sum, op=dist.ReduceOp.SUM, group=self.group)
        return self.world

    def launch(self, tensors):
        """Starts the sum over replicas of every tensor in ``tensors`` (in place)."""
        if self.world <= 1:
            return
        import torch.distributed as dist
        for t in tensors:
            self._pending.append(dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group, async_op=True))

    def finish(self):
        """Returns once every launched reduction is ordered before what the caller does next."""
        for work in self._pending:
            work.wait()
        self._pending = []
