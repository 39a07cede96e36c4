"""The N > 1 protocol of bench.py (replicas, barrier, max-over-ranks timing) on two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_17818_b200 import replicas


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world() == world
        replicas.barrier()
        ms = 10.0 + 5.0 * rank                               # rank 1 is the slow one
        slowest = replicas.max_over_ranks(ms)
        rate = replicas.whole_job_rate(units_per_rank_per_step=1000, steps=4, total_ms_this_rank=ms)
        out.put((rank, slowest, rate))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate in results:
        assert slowest == 15.0                                # max over ranks, on every rank
        assert abs(rate - 2 * 1000 * 4 / 15e-3) < 1e-6        # both replicas' units over the slowest rank's time
    assert [r[0] for r in results] == [0, 1]


def test_single_process_is_its_own_job():
    assert replicas.world() == 1
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(100, 2, 4.0) == 100 * 2 / 4e-3
