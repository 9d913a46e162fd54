"""Host-side logic of the multi-GPU mode.  The PSA forward path has no exchange step, so N GPUs run
N independent replicas of the call; the only communication is the timing reduction (max over ranks).
Works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import os
import subprocess
import sys
from typing import Dict, List, Optional, Sequence

import torch
import torch.distributed as dist


def world_info():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def max_over_ranks(value: float, device=None) -> float:
    """Slowest replica's time: all-reduce MAX (identity when not distributed)."""
    rank, world = world_info()
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_replica: float, ms_local: float, device=None):
    """Whole-job throughput of independent replicas: (world * units) / (slowest replica's time).
    Returns (units per second, ms of the slowest replica)."""
    _, world = world_info()
    ms = max_over_ranks(ms_local, device)
    return world * units_per_replica / (ms * 1e-3), ms


def shard_heads(n_heads: int, rank: int, world: int):
    """Contiguous head range of one rank for a head-sharded call (heads are independent problems)."""
    base, rem = divmod(n_heads, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def rank_env(rank: int, world: int, port: int, base: Optional[Dict[str, str]] = None) -> Dict[str, str]:
    """Environment of one rank of a single-node job: the variables torch.distributed's env:// rendezvous
    reads (one process per GPU: LOCAL_RANK == RANK), on the loopback address."""
    env = dict(os.environ if base is None else base)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "LOCAL_WORLD_SIZE": str(world),
                "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    return env


def free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_ranks(argv: Sequence[str], world: int, port: Optional[int] = None, timeout: Optional[float] = None) -> List[int]:
    """Starts ``world`` copies of ``python argv...``, one per rank, and waits for all of them.  Rank 0
    inherits stdout (it prints the result line); the return codes come back in rank order.  If one
    rank fails the others are terminated (by their own process handles)."""
    port = port or free_port()
    procs = [subprocess.Popen([sys.executable] + list(argv), env=rank_env(r, world, port),
                              stdout=None if r == 0 else subprocess.DEVNULL) for r in range(world)]
    codes: List[Optional[int]] = [None] * world
    try:
        for r, pr in enumerate(procs):
            codes[r] = pr.wait(timeout=timeout)
            if codes[r] != 0:
                break
    finally:
        for r, pr in enumerate(procs):
            if pr.poll() is None:
                pr.terminate()
                try:
                    pr.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    pr.kill()
            if codes[r] is None:
                codes[r] = pr.returncode if pr.returncode is not None else -1
    return [int(c) for c in codes]
