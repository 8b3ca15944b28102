"""Stream sharding over ranks: the only multi-GPU logic of the path.

Frames of one stream depend on each other through the cache, streams are independent, so each
rank (one process per GPU) owns a contiguous set of streams and no data crosses GPUs.  The only
communication is the reduction of the measured time (maximum over ranks).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_streams(rank: int, world: int, streams_per_gpu: int) -> list[int]:
    """Global stream indices owned by ``rank`` (weak scaling: every rank gets ``streams_per_gpu``)."""
    if not (0 <= rank < world) or streams_per_gpu < 1:
        raise ValueError("bad rank / world / streams_per_gpu")
    return list(range(rank * streams_per_gpu, (rank + 1) * streams_per_gpu))


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of ``value`` over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Whole-job throughput: units processed by all ranks over the slowest rank's time."""
    return units_per_rank * world / seconds_max
