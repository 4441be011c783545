"""Replica bookkeeping for runs on more than one GPU.

The path does not shard: sequences are independent, so N GPUs run N independent replicas of the
same verify step with no exchange on the data path.  The only collective traffic is the barrier
around the timed region and the maximum of the ranks' step times; the whole-job throughput is the
positions all replicas scored divided by that slowest time.
"""
from __future__ import annotations

import os


def rank_env():
    """(rank, world_size, local_rank) from the launcher's environment (single process: 0, 1, 0)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Slowest rank's value; a plain pass-through for one process."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, batch: int, gamma: int, ms_per_step: float) -> float:
    """Query positions scored per second by all replicas together: every replica scores
    batch * (gamma + 1) positions per verify step, and the job is as slow as its slowest rank."""
    return world * batch * (gamma + 1) / (ms_per_step * 1e-3)
