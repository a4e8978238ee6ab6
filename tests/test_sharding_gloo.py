"""The multi-GPU path on CPU: two gloo ranks shard the rows, accumulate their own sums/counts (the
oracle stands in for the kernels here), all-reduce once, and must reproduce the unsharded Lloyd step."""
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
