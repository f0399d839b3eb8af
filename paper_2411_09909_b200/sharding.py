"""Row sharding of the quantize + GEMM path over ranks (one process per GPU).

Groups (quantize), output rows (GEMM) and heads (attention) are independent, so a layer shards over
token rows with the weight replicated and NO data-path collective: rank r computes rows
[start, start + count) of C from the same rows of A.  torch.distributed is used only to agree on the
slowest rank's time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(total_rows: int, world: int, rank: int, multiple: int = 128):
    """(start, count) of rank's contiguous row shard; shards are multiples of `multiple` rows except the last."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    blocks = -(-total_rows // multiple)
    per, extra = divmod(blocks, world)
    first = rank * per + min(rank, extra)
    n = per + (1 if rank < extra else 0)
    start = min(first * multiple, total_rows)
    stop = min((first + n) * multiple, total_rows)
    return start, stop - start


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the time of the slowest rank); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Whole-job throughput in units per second: all ranks' units over the slowest rank's time."""
    return world * units_per_rank / (slowest_ms * 1e-3)
