"""Host-side plumbing of `bench.py --gpus N`: replicas only.

The replay path runs on one GPU and has no exchange step.  The members of a GRPO group
are independent replays against the same prefix, so N GPUs are N replicas: every rank
holds its own copy of the resident prefix and replays its own members, and the only
cross-rank operation is the MAX over the ranks' timed regions (never on the data path).
"""
import torch


def member_ids(rank, members_per_rank):
    """Members replayed by `rank`: disjoint across ranks, so no two replicas time the same inputs."""
    return [rank * members_per_rank + m for m in range(members_per_rank)]


def max_over_ranks(value, device, world):
    """MAX over ranks of a per-rank scalar (the timed region's duration)."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_step, steps, world, max_ms):
    """Whole-job units per second: what all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank_step * steps / (max_ms * 1e-3)
