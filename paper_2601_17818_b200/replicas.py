"""Multi-GPU plumbing: the path does not shard (every sequence is independent in every stage and the method has no
exchange step), so N GPUs run N independent replicas of the batch.  What ranks share is the timing protocol only:
a barrier on both sides of the timed region and the MAXIMUM of the per-rank device times."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    """Device sync, process-group barrier (if any), device sync."""
    if torch.cuda.is_available():
        torch.cuda.synchronize()
    if world() > 1:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's figure (times are compared, never summed)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: float, steps: int, total_ms_this_rank: float, device=None) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank_per_step * steps` units (weak
    scaling: per-GPU work is fixed) in the time of the slowest rank."""
    ms = max_over_ranks(total_ms_this_rank, device)
    return world() * units_per_rank_per_step * steps / (ms * 1e-3)


def launch_ranks(n: int, argv, env=None) -> int:
    """Starts `n` ranks of `argv` (a script path followed by its arguments) on this node, one per GPU, under
    torch.distributed.run with a loopback rendezvous on a free port, and returns the launcher's exit code.  This is
    what `bench.py --gpus N` does when it is invoked without a torchrun environment."""
    import os
    import socket
    import subprocess
    import sys
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n)}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), *argv]
    return subprocess.call(cmd, env=dict(os.environ if env is None else env))
