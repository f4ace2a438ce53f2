"""Candidate sharding across ranks.  Candidates are independent problems against one timing table,
so the path shards with no data-path collective: each rank solves a contiguous slice.  The only
exchanges are control-plane: a barrier and a MAX reduction of timings."""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence, Tuple


def shard_range(n_total: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice [start, start + count) of ``n_total`` candidates for ``rank``; the first
    ``n_total % world`` ranks take one extra candidate."""
    if world < 1 or not (0 <= rank < world) or n_total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_total, world)
    count = base + (1 if rank < extra else 0)
    start = rank * base + min(rank, extra)
    return start, count


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Aggregate throughput when every rank processed ``units_per_rank`` units (weak scaling) and
    the slowest rank took ``seconds_max``."""
    return world * units_per_rank / seconds_max


def free_port() -> int:
    """A TCP port on 127.0.0.1 that is free right now (for the rendezvous of a local launch)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def launch_command(script: str, script_args: Sequence[str], nproc: int, port: Optional[int] = None) -> List[str]:
    """The command that starts ``nproc`` ranks of ``script`` on this node, one process per rank, with a
    127.0.0.1 rendezvous (the container's hostname may not resolve)."""
    if nproc < 1:
        raise ValueError("need at least one rank")
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(nproc)}",
            "--master-addr", "127.0.0.1", "--master-port", str(port if port is not None else free_port()),
            script, *script_args]


def under_launcher() -> bool:
    """True inside a process that a launcher started as one rank of several (WORLD_SIZE is set)."""
    return "WORLD_SIZE" in os.environ


def spawn_ranks(script: str, script_args: Sequence[str], nproc: int, timeout: Optional[float] = None) -> int:
    """Run ``script`` as ``nproc`` ranks and wait; the ranks inherit stdout/stderr (rank 0 prints the
    result).  Returns the launcher's exit code."""
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "1")
    return subprocess.run(launch_command(script, script_args, nproc), env=env, timeout=timeout).returncode
