"""How the path spreads over several GPUs: by sequence, with no exchange on the data path.

Every step of the method is independent per sequence, and KV-cache compression and decode attention
are independent per (sequence, KV head) (Section 3.2.2, paragraph 2), so N ranks simply run N
replicas on their own sequences.  The only communication is the bookkeeping of a measurement:
a barrier and the maximum of the per-rank step times.  This module holds that host logic so that
it can be exercised with CPU process groups as well.
"""
from __future__ import annotations

from typing import Tuple

import torch

from . import inputs as I


def shard_workload(w: I.Workload, rank: int, world: int) -> I.Workload:
    """The workload rank ``rank`` of ``world`` runs: same shapes (weak scaling), its own sequences."""
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside [0, {world})")
    return w if world == 1 else I.shrink(w, seed=w.seed + 1000 * rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of ``value`` over the ranks of the default process group (the value itself without one)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: int, ms_local: float, world: int, device="cpu") -> Tuple[float, float]:
    """(whole-job units per second, step time in ms): every rank processed ``units_per_rank`` units,
    the job took as long as its slowest rank."""
    ms = max_over_ranks(ms_local, device)
    return units_per_rank * world / (ms * 1e-3), ms
