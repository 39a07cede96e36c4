"""A stand-in for bench.py's GPU arm on the CPU: the same rank protocol (environment from the launcher, gloo process
group, barrier on both sides of the timed region, maximum over ranks, one JSON line from rank 0), with a sleep in place
of the step.  Started by tests/test_replicas_gloo.py through replicas.launch_ranks, the launcher bench.py uses."""
import argparse
import json
import os
import time

import torch.distributed as dist

from paper_2601_17818_b200 import replicas


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--out", required=True)
    args = ap.parse_args()
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    replicas.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.01 * (1 + rank))                       # the higher rank is the slower one
    ms = (time.perf_counter() - t0) * 1e3
    replicas.barrier()
    slowest = replicas.max_over_ranks(ms)
    value = replicas.whole_job_rate(1000, args.steps, ms)
    if rank == 0:
        with open(args.out, "w") as fh:
            json.dump({"n_gpus": world, "gpus_arg": args.gpus, "steps": args.steps, "ms": slowest, "value": value}, fh)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
