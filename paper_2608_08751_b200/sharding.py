"""Sharding over more than one GPU: one process per GPU, torch.distributed for the exchange.

Two ways to split the path (rows are independent; Eq. 1 is a minimum over centroids):

* rows sharded, centroids replicated (``shard_rows``): routing needs no collective.  A Lloyd
  iteration has one exchange: every rank accumulates sums and counts over its own rows, then one
  all-reduce makes them global before each rank finalizes the same new centroids
  (``allreduce_lloyd``).
* centroids sharded, queries replicated (``shard_centroids``, ``route_centroid_split``), for tables
  too large to replicate (Sec. 4.1: N_list up to millions): every rank routes all queries against
  its own slice of the table, the [nq, k] (distance, id) lists are all-gathered, and every rank
  merges them to the k nearest overall -- ties across shards go to the lower global id.

Only plumbing lives here (ranges, id offsets, padding, the torch.distributed calls); routing and
the merge are the library's calls, passed in as functions so that the same plumbing runs in CPU
tests with stand-ins.  No scaling curve has been measured with either split.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(n: int, rank: int, world: int, align: int = 128) -> tuple[int, int]:
    """[begin, end) of this rank's rows: contiguous, balanced, begin aligned to the 128-row tile."""
    per = -(-n // world)
    per = -(-per // align) * align
    begin = min(n, rank * per)
    return begin, min(n, begin + per)


def shard_centroids(nlist: int, rank: int, world: int, align: int = 256) -> tuple[int, int]:
    """[begin, end) of this rank's centroids: contiguous, balanced, begin aligned to the centroid tile."""
    return shard_rows(nlist, rank, world, align)


def allreduce_lloyd(sums: torch.Tensor, counts: torch.Tensor) -> None:
    """In-place sum of the per-rank Lloyd accumulators over the default process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
        dist.all_reduce(counts, op=dist.ReduceOp.SUM)


def pad_shard_lists(ids: torch.Tensor, dists: torch.Tensor, k: int, id_offset: int):
    """Local lists [nq, k_local] -> [nq, k] with global ids; unused places hold (+inf, int32 max)."""
    nq, kl = ids.shape
    out_ids = torch.full((nq, k), torch.iinfo(torch.int32).max, dtype=torch.int32, device=ids.device)
    out_d = torch.full((nq, k), float("inf"), dtype=torch.float32, device=ids.device)
    out_ids[:, :kl] = ids + id_offset
    out_d[:, :kl] = dists
    return out_ids, out_d


def route_centroid_split(queries: torch.Tensor, centroid_shard: torch.Tensor, id_offset: int, k: int,
                         route_fn, merge_fn, group=None):
    """Routing against a table split over the ranks of `group`.

    queries [nq, d] (the same on every rank), centroid_shard [nlist_r, d]: this rank's slice, whose
    first row has global id `id_offset`.  route_fn(queries, shard, k_local) -> (ids [nq, k_local] int32,
    dists [nq, k_local] float32), local ids, ascending; merge_fn(shard_ids [world, nq, k], shard_dists
    [world, nq, k]) -> (ids [nq, k], dists [nq, k]).  Returns the merged lists (identical on every rank).
    """
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    k_local = min(k, centroid_shard.shape[0])
    ids, dists = route_fn(queries, centroid_shard, k_local)
    ids, dists = pad_shard_lists(ids, dists, k, id_offset)
    if world == 1:
        return merge_fn(ids.unsqueeze(0).contiguous(), dists.unsqueeze(0).contiguous())
    nq = ids.shape[0]
    all_ids = torch.empty((world * nq, k), dtype=ids.dtype, device=ids.device)  # rank-major concatenation
    all_d = torch.empty((world * nq, k), dtype=dists.dtype, device=dists.device)
    dist.all_gather_into_tensor(all_ids, ids.contiguous(), group=group)
    dist.all_gather_into_tensor(all_d, dists.contiguous(), group=group)
    return merge_fn(all_ids.view(world, nq, k), all_d.view(world, nq, k))
