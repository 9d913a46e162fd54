"""Host-side logic of the multi-GPU mode.  The PSA forward path has no exchange step, so N GPUs run
N independent replicas of the call; the only communication is the timing reduction (max over ranks).
Works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

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
