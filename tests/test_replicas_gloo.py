"""Two CPU ranks over gloo: the multi-GPU bookkeeping of bench.py (replicas, no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_08600_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.rank_env() == (rank, world, rank)
    ms_local = 3.0 + rank                                   # rank 1 is the slow replica
    dist.barrier()
    ms = replicas.max_over_ranks(ms_local, world)
    value = replicas.whole_job_tokens_per_s(world, 1, 5, ms)
    out.put((rank, ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 4.0                                    # the maximum over ranks, on every rank
        assert abs(value - 2 * 6 / 4.0e-3) < 1e-9           # two replicas x 6 positions per slowest step


def test_single_process_passthrough():
    assert replicas.max_over_ranks(2.5, 1) == 2.5
    assert replicas.whole_job_tokens_per_s(1, 16, 5, 10.0) == 9600.0


_CHILD = """
import torch.distributed as dist
from paper_2505_08600_b200 import replicas
rank, world, local = replicas.rank_env()
dist.init_process_group('gloo')
ms = replicas.max_over_ranks(2.0 + 3.0 * rank, world)
if rank == 0:
    print('slowest', ms, replicas.whole_job_tokens_per_s(world, 1, 5, ms))
else:
    print('not rank 0')
dist.barrier()
dist.destroy_process_group()
"""


def test_spawn_local_launches_the_ranks_and_returns_rank_zero_output():
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    rc, out = replicas.spawn_local(2, [sys.executable, "-c", f"import sys; sys.path.insert(0, {root!r})\n" + _CHILD], timeout=180)
    assert rc == 0
    assert out.split() == ["slowest", "5.0", str(2 * 6 / 5.0e-3)]


def test_spawn_local_reports_a_failing_rank():
    import sys
    rc, out = replicas.spawn_local(2, [sys.executable, "-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"], timeout=60)
    assert rc == 3 and out == ""
