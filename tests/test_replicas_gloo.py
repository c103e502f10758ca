"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on CPU with gloo."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2102_08374_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local = 0.010 * (rank + 1)                     # rank 1 is the slow one
        dist.barrier()
        slow = replicas.max_over_ranks(dist, local)
        thr = replicas.whole_job_throughput(dist, 1000, local)
        out.put((rank, slow, thr, replicas.rank_seed_base(rank)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, thr, seed in got:
        assert slow == pytest.approx(0.020)
        assert thr == pytest.approx(2 * 1000 / 0.020)
    assert got[0][3] != got[1][3]


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(None, 1.5) == 1.5
    assert replicas.whole_job_throughput(None, 10, 2.0) == 5.0
