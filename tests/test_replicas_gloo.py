"""CPU, two processes over gloo: the rank bookkeeping of a multi-GPU run (replicas only: no data-path collective).

What N > 1 adds to a measurement is only this: barriers around the timed region, the job's duration as the
maximum over the ranks, and the job's throughput as the sum of the replicas' work over that duration.
"""
import os
import socket

import pytest


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    import torch.distributed as dist
    from paper_2408_11743_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        mine = 0.5 * (rank + 1)                      # rank 1 is the slow one
        job = replicas.max_over_ranks(mine)
        value = replicas.job_throughput(units_per_rank=100.0, world=world, job_seconds=job)
        replicas.barrier()
        out.put((rank, job, value))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, job, value in results:
        assert job == pytest.approx(1.0)             # max(0.5, 1.0) on every rank
        assert value == pytest.approx(200.0)         # 2 replicas x 100 units / 1 s


def test_single_process_needs_no_process_group():
    from paper_2408_11743_b200 import replicas
    assert replicas.max_over_ranks(0.25) == 0.25
    assert replicas.job_throughput(10.0, 1, 0.5) == 20.0
    replicas.barrier()
