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


def _free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_local(n: int, argv, timeout: float | None = None):
    """Runs `argv` (a command line) as n rank processes of one node, the way a launcher would: RANK, LOCAL_RANK,
    WORLD_SIZE and a rendezvous on 127.0.0.1 in the environment.  Rank 0's stdout is captured and returned; the other
    ranks' stdout is dropped and every rank's stderr is passed through.  Returns (worst exit code, rank 0's stdout)."""
    import subprocess
    port = _free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env, stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, worst = "", 0
    try:
        out, _ = procs[0].communicate(timeout=timeout)
        for p in procs:
            p.wait(timeout=timeout)
    except subprocess.TimeoutExpired:
        worst = 124
    finally:
        for p in procs:                  # the exact processes started above, nothing else
            if p.poll() is None:
                p.kill()
                p.wait()
    for p in procs:
        if p.returncode != 0:
            worst = worst or p.returncode
    return worst, out
