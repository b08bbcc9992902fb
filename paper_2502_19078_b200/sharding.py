"""Host-side logic of multi-GPU runs: the path partitions over independent sequences (each has its own
scores, thresholds and masks), so ranks share nothing on the data path.  What is left is bookkeeping:
which sequences a rank owns, and the whole-job rate = all ranks' units / the slowest rank's time."""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_range(n_units: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced [lo, hi) of n_units for this rank (sizes differ by at most one)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside [0, world)")
    return (n_units * rank) // world, (n_units * (rank + 1)) // world


def shard_sizes(n_units: int, world: int) -> List[int]:
    return [shard_range(n_units, r, world)[1] - shard_range(n_units, r, world)[0] for r in range(world)]


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time (or any per-rank scalar's maximum); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_this_rank: float, elapsed_ms_this_rank: float, device="cpu") -> Tuple[float, float]:
    """(units of all ranks per second, the slowest rank's milliseconds)."""
    ms = max_over_ranks(elapsed_ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def under_launcher() -> bool:
    """True when this process was started as one rank of a multi-process job (torchrun or launch_ranks)."""
    import os
    return "RANK" in os.environ and "WORLD_SIZE" in os.environ


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n_ranks: int, argv: List[str], devices_available: int | None = None, timeout_s: float | None = None,
                 extra_env: dict | None = None) -> int:
    """Start n_ranks copies of `python argv...` on this node, one per GPU, with RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_ADDR / MASTER_PORT set as torchrun would, wait for all of them and return the worst exit code.
    Rank 0 inherits stdout (it prints the result line); every rank inherits stderr.  Refuses more ranks than
    devices.  If a rank fails, the others are terminated (by their own PIDs)."""
    import os
    import subprocess
    import sys
    import time
    if n_ranks < 1:
        raise ValueError("n_ranks must be at least 1")
    if devices_available is not None and n_ranks > devices_available:
        raise ValueError(f"--gpus {n_ranks} asks for more devices than this node has ({devices_available})")
    port = free_port()
    procs = []
    for r in range(n_ranks):
        env = dict(os.environ)
        env.update({"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n_ranks), "LOCAL_WORLD_SIZE": str(n_ranks),
                    "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        env.setdefault("NCCL_DEBUG", "WARN")
        if extra_env:
            env.update(extra_env)
        procs.append(subprocess.Popen([sys.executable] + list(argv), env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    deadline = None if timeout_s is None else time.monotonic() + timeout_s
    worst = 0
    pending = list(procs)
    while pending:
        for p in list(pending):
            rc = p.poll()
            if rc is None:
                continue
            pending.remove(p)
            if rc != 0:
                worst = worst or rc
                for q in pending:      # a failed rank leaves the others waiting at a collective: stop them
                    q.terminate()
        if deadline is not None and time.monotonic() > deadline:
            for q in pending:
                q.terminate()
            worst = worst or 124
            deadline = None
        time.sleep(0.05)
    return worst
