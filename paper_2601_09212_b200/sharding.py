"""Data-parallel use of the verify step: sequences are independent, so a batch is cut into
contiguous shards, one per rank, and nothing is exchanged on the data path.  Only timing is
reduced across ranks (maximum), with ``torch.distributed`` as the plumbing."""
from __future__ import annotations

from typing import Tuple


def shard_bounds(n_sequences: int, world_size: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the sequences rank ``rank`` verifies: contiguous, sizes differing by at most one."""
    if world_size < 1 or not 0 <= rank < world_size or n_sequences < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_sequences, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of ``value`` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world_size: int, seconds_max: float) -> float:
    """Whole-job rate when every rank processed ``units_per_rank`` units and the slowest took ``seconds_max``."""
    return units_per_rank * world_size / seconds_max
