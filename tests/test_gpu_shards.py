"""Centroid-split routing on one GPU: the shards are routed one after the other on the same device
(no rank waits for another), gathered into the [parts, nq, k] layout an all-gather would give, and
merged by ivf_merge_shards.  Checked against the oracle on the whole table."""
import numpy as np
import pytest
import torch

from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import sharding, synth

import parity

pytestmark = pytest.mark.gpu


def _split_route(q, c, k, parts):
    qt = torch.from_numpy(q).cuda()
    all_ids, all_d = [], []
    for r in range(parts):
        b, e = sharding.shard_centroids(c.shape[0], r, parts)
        shard = torch.from_numpy(np.ascontiguousarray(c[b:e])).cuda()
        kl = min(k, e - b)
        if kl == 1:
            ids, d = B.ivf_assign(qt, shard)
            ids, d = ids.view(-1, 1), d.view(-1, 1)
        else:
            ids, d = B.ivf_route(qt, shard, kl)
        ids, d = sharding.pad_shard_lists(ids, d, k, b)
        all_ids.append(ids)
        all_d.append(d)
    ids, d = B.ivf_merge_shards(torch.stack(all_ids).contiguous(), torch.stack(all_d).contiguous())
    B.ivf_check()
    return ids.cpu().numpy(), d.cpu().numpy()


@pytest.mark.parametrize("n,nlist,d,k,parts,dtype", [(300, 3000, 128, 40, 2, "u8"), (130, 5000, 96, 17, 3, "f32"),
                                                     (64, 600, 64, 100, 2, "f32"), (200, 9000, 128, 512, 4, "u8"),
                                                     (77, 2000, 32, 1, 2, "f32")])
def test_split_routing_matches_oracle(n, nlist, d, k, parts, dtype):
    rng = np.random.default_rng(n + nlist)
    if dtype == "u8":
        x = rng.integers(0, 256, (n, d)).astype(np.uint8)
        c = (rng.standard_normal((nlist, d)) * 40 + 100).astype(np.float32)
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
        c = rng.standard_normal((nlist, d)).astype(np.float32)
    ids, dists = _split_route(x, c, k, parts)
    parity.check_route(x, c, k, ids, dists)


def test_split_routing_integer_ties_across_shards_bit_exact():
    q, c = synth.integer_case(200, 3000, 64, seed=9)
    c[2999] = c[3]        # equal centroids in different shards: the lower global id must win
    c[1700] = c[100]
    ids, dists = _split_route(q, c, 50, 3)
    parity.check_route(q, c, 50, ids, dists, exact=True)


def test_merge_kernel_against_lexsort():
    rng = np.random.default_rng(3)
    parts, nq, k = 5, 300, 64
    d = np.sort(rng.integers(0, 50, (parts, nq, k)).astype(np.float32), axis=2)  # many equal distances
    d[4, :, 40:] = np.inf                                                        # a short shard
    ids = rng.permutation(parts * nq * k).astype(np.int32).reshape(parts, nq, k)
    # each list ascending by (distance, id)
    order = np.lexsort((ids, d), axis=2)
    ids, d = np.take_along_axis(ids, order, 2), np.take_along_axis(d, order, 2)
    g_ids, g_d = B.ivf_merge_shards(torch.from_numpy(ids).cuda(), torch.from_numpy(d).cuda())
    B.ivf_check()
    fi, fd = ids.transpose(1, 0, 2).reshape(nq, -1), d.transpose(1, 0, 2).reshape(nq, -1)
    o = np.lexsort((fi, fd), axis=1)[:, :k]
    assert (g_ids.cpu().numpy() == np.take_along_axis(fi, o, 1)).all()
    assert (g_d.cpu().numpy() == np.take_along_axis(fd, o, 1)).all()
