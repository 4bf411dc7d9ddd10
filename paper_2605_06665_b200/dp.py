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
