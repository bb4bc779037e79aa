"""Host-side helpers for running the path on several GPUs of one node.

Rows (tokens) are independent in every step of the path, so scale-out is plain sharding of M
with the weights replicated: no data-path collective.  torch.distributed is used only to agree
on a time (max over ranks) and for barriers.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
import tempfile
import time
from typing import List, Optional, Sequence, Tuple


def row_shard(M: int, rank: int, world: int, align: int = 1) -> Tuple[int, int]:
    """[begin, end) of the rows rank `rank` owns when M rows are split over `world` ranks in
    contiguous pieces whose sizes differ by less than 2 * `align` rows (pieces are multiples of
    `align` except possibly the last)."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank / world size")
    units = (M + align - 1) // align
    base, extra = divmod(units, world)
    begin_u = rank * base + min(rank, extra)
    end_u = begin_u + base + (1 if rank < extra else 0)
    return min(begin_u * align, M), min(end_u * align, M)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank number over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job rate: every rank processed `units_per_rank` in `ms` (already the max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def rank_environment(rank: int, world: int, port: int, base: Optional[dict] = None) -> dict:
    """Environment of one rank of a single-node job: what a torchrun launch would have set."""
    env = dict(os.environ if base is None else base)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), LOCAL_WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    return env


def spawn_ranks(world: int, argv: Sequence[str], timeout: Optional[float] = None) -> Tuple[int, str]:
    """Runs `argv` (a command line) as `world` processes of one node, one per rank, each with the
    rendezvous variables of `rank_environment`.  Rank 0's standard output is captured and returned;
    the other ranks' output goes to this process's stderr.  Returns (worst exit code, rank 0's stdout).
    A rank that fails or overruns `timeout` seconds ends the others (by PID)."""
    if world < 1:
        raise ValueError("world size must be positive")
    port = free_port()
    out_file = tempfile.TemporaryFile(mode="w+")
    procs: List[subprocess.Popen] = []
    for rank in range(world):
        procs.append(subprocess.Popen(list(argv), env=rank_environment(rank, world, port),
                                      stdout=out_file if rank == 0 else sys.stderr))
    # Rank 0's output goes to a temporary file (no pipe to fill up); all children are polled, and the first failure or the
    # deadline ends the others, so that a rank lost before a collective cannot leave the rest waiting for ever.
    worst, out0 = 0, ""
    deadline = None if timeout is None else time.monotonic() + timeout
    try:
        while True:
            codes = [p.poll() for p in procs]
            failed = [c for c in codes if c not in (None, 0)]
            if failed:
                worst = failed[0]
                break
            if all(c == 0 for c in codes):
                break
            if deadline is not None and time.monotonic() > deadline:
                worst = 124
                break
            time.sleep(0.05)
    finally:
        for p in procs:
            if p.poll() is None:
                p.kill()
                p.wait()
        out_file.seek(0)
        out0 = out_file.read()
        out_file.close()
    return worst, out0
