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


def test_launcher_starts_the_ranks_itself(tmp_path):
    """`bench.py --gpus N` invoked plainly re-launches itself through replicas.launch_ranks; here the same launcher
    starts two CPU ranks of a stub step and rank 0 reports the whole job."""
    import json
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    out = tmp_path / "line.json"
    env = dict(os.environ, PYTHONPATH=os.pathsep.join([os.path.dirname(here)] + sys.path))
    rc = replicas.launch_ranks(2, [os.path.join(here, "replica_stub.py"), "--gpus", "2", "--steps", "3", "--out", str(out)],
                               env=env)
    assert rc == 0
    line = json.loads(out.read_text())
    assert line["n_gpus"] == 2 and line["gpus_arg"] == 2
    assert line["ms"] >= 3 * 0.01 * 2 * 1e3 * 0.9            # the slower rank's time
    assert abs(line["value"] - 2 * 1000 * 3 / (line["ms"] * 1e-3)) / line["value"] < 0.35


def test_bench_relaunches_itself_when_asked_for_several_gpus(monkeypatch):
    import importlib.util
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    seen = {}
    monkeypatch.setattr(replicas, "launch_ranks", lambda n, argv, env=None: seen.update(n=n, argv=argv) or 0)
    monkeypatch.delenv("RANK", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7"])
    try:
        bench.main()
    except SystemExit as e:
        assert e.code == 0
    assert seen["n"] == 4 and seen["argv"][1:] == ["--gpus", "4", "--steps", "7"]
    assert seen["argv"][0].endswith("bench.py")
