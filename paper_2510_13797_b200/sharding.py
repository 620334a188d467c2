"""Host-side logic of the multi-GPU runs: one process per GPU, sequences sharded, no exchange.

Sequences are independent units (each has its own cache, ratio and page table), so a batch is
partitioned across ranks and every rank runs the whole hot path on its shard with its own pool and
free stack.  Nothing of the data path crosses GPUs; the only communication is the reduction of
the measured times (the slowest rank defines the time of the job) and of unit counts.
Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard_range(n_units: int, world: int, rank: int) -> range:
    """Contiguous, balanced shard of n_units independent units: sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError(f"rank {rank} outside world {world}")
    per, rem = divmod(n_units, world)
    start = rank * per + min(rank, rem)
    return range(start, start + per + (1 if rank < rem else 0))


def rank_seed_offset(seed: int, rank: int) -> int:
    """Weak scaling: every rank runs the same shapes on its own seeded inputs."""
    return seed + rank


def _reduce(values: Sequence[float], op, device) -> List[float]:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return [float(x) for x in t]


def max_over_ranks(values: Sequence[float], device="cpu") -> List[float]:
    """Element-wise maximum of per-rank measurements (times): the slowest rank counts."""
    return _reduce(values, dist.ReduceOp.MAX, device)


def sum_over_ranks(values: Sequence[float], device="cpu") -> List[float]:
    """Element-wise sum of per-rank counts (units processed)."""
    return _reduce(values, dist.ReduceOp.SUM, device)


def job_throughput(units_all_ranks: float, ms_max: float) -> float:
    """Whole-job throughput: the units every rank processed, over the slowest rank's time."""
    return units_all_ranks / (ms_max * 1e-3)
