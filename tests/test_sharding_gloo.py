"""The multi-GPU paths on CPU (the oracle and numpy stand in for the kernels here).  Row split: two gloo
ranks shard the rows, accumulate their own sums/counts, all-reduce once, and must reproduce the
unsharded Lloyd step.  Centroid split: two ranks route all queries against their own slice of the
table, all-gather the lists, merge by (distance, id), and must reproduce the unsharded routing."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle
from paper_2608_08751_b200 import sharding, synth


def test_shard_rows_partition():
    for n, w in [(1000, 2), (128, 4), (1, 3), (100000, 8), (257, 2)]:
        spans = [sharding.shard_rows(n, r, w) for r in range(w)]
        assert spans[0][0] == 0 and spans[-1][1] == n
        for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(b % 128 == 0 or b == n for b, _ in spans)


def _worker(rank, world, port, n, nlist, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = synth.sift_like_rows(2, rows=n)
    c = synth.sift_like_centroids(nlist)
    b, e = sharding.shard_rows(n, rank, world)
    ids, _ = oracle.assign(x[b:e], c)
    s, cnt, ok = oracle.update(x[b:e], ids, nlist)
    sums, counts = torch.from_numpy(s.astype(np.float32)), torch.from_numpy(cnt)
    sharding.allreduce_lloyd(sums, counts)
    new_c = oracle.finalize(sums.numpy().astype(np.float64), counts.numpy(), c)
    if rank == 0:
        np.save(out, new_c)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_lloyd_step_equals_unsharded(tmp_path):
    n, nlist = 3000, 40
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "c.npy")
    mp.spawn(_worker, args=(2, port, n, nlist, out), nprocs=2, join=True)
    x = synth.sift_like_rows(2, rows=n)
    c = synth.sift_like_centroids(nlist)
    ids, _ = oracle.assign(x, c)
    s, cnt, _ = oracle.update(x, ids, nlist)
    want = oracle.finalize(s, cnt, c)
    got = np.load(out)
    assert (got == want).all()  # uint8 rows: sums are exact integers in fp32, so the result is identical


def _route_stub(queries, shard, k):
    ids, d, _ = oracle.route(queries.numpy(), shard.numpy(), k)
    return torch.from_numpy(ids), torch.from_numpy(d.astype(np.float32))


def _merge_stub(all_ids, all_d):
    # the k smallest by (distance, id) over the gathered lists
    world, nq, k = all_ids.shape
    ids = all_ids.permute(1, 0, 2).reshape(nq, world * k).numpy()
    d = all_d.permute(1, 0, 2).reshape(nq, world * k).numpy()
    order = np.lexsort((ids, d), axis=1)[:, :k]
    return torch.from_numpy(np.take_along_axis(ids, order, 1)), torch.from_numpy(np.take_along_axis(d, order, 1))


def _split_inputs(nlist):
    rng = np.random.default_rng(5)
    q = rng.integers(0, 4, (60, 16)).astype(np.float32)       # few distinct values: many exact ties,
    c = rng.integers(0, 4, (nlist, 16)).astype(np.float32)    # also across the shard boundary
    c[nlist - 1] = c[0]
    c[300] = c[200]
    return q, c


def _split_worker(rank, world, port, nlist, k, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, c = _split_inputs(nlist)
    b, e = sharding.shard_centroids(nlist, rank, world)
    ids, d = sharding.route_centroid_split(torch.from_numpy(q), torch.from_numpy(c[b:e].copy()), b, k,
                                           _route_stub, _merge_stub)
    np.save(out + f".{rank}.ids.npy", ids.numpy())
    np.save(out + f".{rank}.d.npy", d.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_shard_centroids_partition():
    for nlist, w in [(1000, 2), (65536, 8), (300, 4), (257, 2)]:
        spans = [sharding.shard_centroids(nlist, r, w) for r in range(w)]
        assert spans[0][0] == 0 and spans[-1][1] == nlist
        assert all(a1 == b0 for (_, a1), (b0, _) in zip(spans, spans[1:]))


def test_two_rank_centroid_split_equals_unsharded(tmp_path):
    # 600 centroids over 2 ranks (512 + 88): the second shard has fewer centroids than k, so its list
    # is padded; duplicated centroids sit in different shards, so ties cross the shard boundary
    nlist, k = 600, 100
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "split")
    mp.spawn(_split_worker, args=(2, port, nlist, k, out), nprocs=2, join=True)
    q, c = _split_inputs(nlist)
    o_ids, o_d, _ = oracle.route(q, c, k)
    for rank in range(2):
        ids, d = np.load(out + f".{rank}.ids.npy"), np.load(out + f".{rank}.d.npy")
        assert (ids == o_ids).all()                      # ties resolved to the lower global id
        assert (d == o_d.astype(np.float32)).all()       # small integers: exact in fp32
