"""Row sharding for more than one GPU: rows are independent, centroids are replicated.

Routing needs no collective.  A Lloyd iteration has one exchange: every rank accumulates sums and
counts over its own rows, then one all-reduce makes them global before each rank finalizes the
same new centroids.  Only plumbing lives here (ranges and the torch.distributed call)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(n: int, rank: int, world: int, align: int = 128) -> tuple[int, int]:
    """[begin, end) of this rank's rows: contiguous, balanced, begin aligned to the 128-row tile."""
    per = -(-n // world)
    per = -(-per // align) * align
    begin = min(n, rank * per)
    return begin, min(n, begin + per)


def allreduce_lloyd(sums: torch.Tensor, counts: torch.Tensor) -> None:
    """In-place sum of the per-rank Lloyd accumulators over the default process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
        dist.all_reduce(counts, op=dist.ReduceOp.SUM)
