"""Seeded random sweeps over shapes, element types and k for every entry point, each case compared
with the CPU oracle: the fixed parity cases pick the sizes someone thought of, these pick the rest."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _points(rng, dtype, n, d, integer):
    if dtype == "u8":
        return rng.integers(0, 16 if integer else 256, (n, d)).astype(np.uint8)
    if dtype == "i8":
        return rng.integers(-8 if integer else -128, 8 if integer else 128, (n, d)).astype(np.int8)
    return (rng.standard_normal((n, d)) * rng.choice([1e-3, 1.0, 50.0])).astype(np.float32)


def _centroids(rng, dtype, nlist, d, integer):
    if integer:
        lo, hi = (0, 16) if dtype == "u8" else (-8, 8)
        return rng.integers(lo, hi, (nlist, d)).astype(np.float32)
    if dtype == "u8":
        return (rng.standard_normal((nlist, d)) * 40 + 100).astype(np.float32)
    if dtype == "i8":
        return (rng.standard_normal((nlist, d)) * 40).astype(np.float32)
    return (rng.standard_normal((nlist, d))).astype(np.float32)


@pytest.mark.parametrize("seed", range(40))
def test_route_random_shapes(seed):
    rng = np.random.default_rng(5000 + seed)
    dtype = rng.choice(["u8", "i8", "f32"])
    integer = dtype != "f32" and rng.random() < 0.4
    d = int(rng.choice([4, 8, 16, 20, 32, 48, 64, 96, 100, 128, 160, 192, 256]))
    n = int(rng.choice([1, 2, 31, 127, 128, 129, 255, 257, 500, 1000, 1500]))
    nlist = int(rng.choice([1, 2, 7, 64, 255, 256, 257, 1000, 4096, 9000, 20000, 70000]))
    k = int(min(nlist, rng.choice([1, 1, 2, 3, 10, 16, 17, 50, 64, 100, 200, 512])))
    if n * nlist * d > 3e9:  # keep the oracle quick
        n = max(1, int(3e9 / (nlist * d)))
    x = _points(rng, dtype, n, d, integer)
    c = _centroids(rng, dtype, nlist, d, integer)
    if k == 1 and rng.random() < 0.5:
        ids, dists = B.ivf_assign(_t(x), _t(c))
    else:
        ids, dists = B.ivf_route(_t(x), _t(c), k)
    B.ivf_check()
    parity.check_route(x, c, k, ids.cpu().numpy(), dists.cpu().numpy(), exact=bool(integer))


@pytest.mark.parametrize("seed", range(12))
def test_update_and_reorder_random_shapes(seed):
    rng = np.random.default_rng(6000 + seed)
    dtype = rng.choice(["u8", "i8", "f32"])
    d = int(rng.choice([4, 16, 36, 100, 128, 256]))
    n = int(rng.choice([1, 100, 5000, 40000]))
    nlist = int(rng.choice([1, 3, 300, 5000, 70000]))
    x = _points(rng, dtype, n, d, False)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    # accumulation on top of earlier sums: integers for byte-typed points (the result stays exact)
    base = rng.integers(-50, 50, (nlist, d)) if dtype != "f32" else rng.standard_normal((nlist, d))
    sums = torch.from_numpy(base.astype(np.float32)).cuda()
    counts = torch.from_numpy(rng.integers(0, 5, nlist).astype(np.int64)).cuda()
    base_s, base_c = sums.cpu().numpy().astype(np.float64), counts.cpu().numpy().copy()
    B.ivf_centroid_update(_t(x), _t(ids), sums, counts)
    B.ivf_check()
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy(), base_s, base_c)
    xr, offsets, order = B.ivf_cluster_major_reorder(_t(x), _t(ids), nlist)
    B.ivf_check()
    want_off, _ = O.reorder(ids, nlist)
    order = order.cpu().numpy()
    assert (offsets.cpu().numpy() == want_off).all()
    assert (np.sort(order) == np.arange(n)).all() and (np.diff(ids[order]) >= 0).all()
    assert (xr.cpu().numpy() == x[order]).all()


@pytest.mark.parametrize("seed", range(16))
def test_pq_random_shapes(seed):
    rng = np.random.default_rng(7000 + seed)
    dtype = rng.choice(["u8", "i8", "f32"])
    pq_m, dsub = [(32, 4), (16, 8), (32, 3), (16, 6), (20, 5), (50, 2), (8, 1), (1, 16), (64, 2), (4, 7)][seed % 10]
    d = pq_m * dsub
    nlist = int(rng.choice([3, 40, 400]))
    n = int(rng.choice([200, 5000, 30000]))
    nq = int(rng.choice([1, 7, 40]))
    nprobe = int(min(nlist, rng.choice([1, 3, 16, 64])))
    n_rerank = int(rng.choice([1, 10, 100, 512, 1024]))
    c = _centroids(rng, dtype, nlist, d, False)
    ids, offsets = synth.skewed_list_ids(n, nlist, seed=seed, sigma=float(rng.choice([0.3, 1.0, 2.0])))
    x = _points(rng, dtype, n, d, False)
    cb = synth.pq_codebooks(pq_m, dsub, 20.0 if dtype != "f32" else 0.5, seed=seed, integer=bool(rng.random() < 0.3))
    q = _points(rng, dtype, nq, d, False)
    probes = synth.distinct_probes(nq, nlist, nprobe, seed=seed)
    want_codes = O.pq_encode(x, ids, c, cb)
    got_codes = B.ivf_pq_encode(_t(x), _t(ids), _t(c), _t(cb))
    B.ivf_check()
    assert (got_codes.cpu().numpy() == want_codes).all()
    want = O.pq_search(q, c, probes, offsets, want_codes, cb, n_rerank)
    got = B.ivf_pq_search(_t(q), _t(c), _t(probes), _t(offsets), _t(want_codes), _t(cb), n_rerank)
    B.ivf_check()
    assert (got[0].cpu().numpy() == want[0]).all() and (got[2].cpu().numpy() == want[2]).all()
    assert (got[1].cpu().numpy().view(np.uint32) == want[1].view(np.uint32)).all()


@pytest.mark.parametrize("seed", range(8))
def test_candidates_random_shapes(seed):
    rng = np.random.default_rng(8000 + seed)
    dtype = rng.choice(["u8", "i8", "f32"])
    d = int(rng.choice([4, 36, 100, 128, 256]))
    n, nlist, m = int(rng.choice([1, 333, 4000])), int(rng.choice([1, 50, 3000])), int(rng.choice([1, 2, 3, 8, 11]))
    x = _points(rng, dtype, n, d, True)
    c = _centroids(rng, dtype, nlist, d, True)
    cand = rng.integers(0, nlist, (n, m)).astype(np.int32)
    ids, dist = B.ivf_assign_candidates(_t(x), _t(c), _t(cand))
    B.ivf_check()
    want_ids, want_d = O.assign_candidates(x, c, cand)
    ids, dist = ids.cpu().numpy(), dist.cpu().numpy().astype(np.float64)
    if dtype != "f32":  # integer data: exact
        assert (ids == want_ids).all() and (dist == want_d).all()
    else:
        true_d = O.pair_dists(x, c, np.arange(n), ids)
        assert np.allclose(dist, true_d, rtol=1e-5, atol=1e-30)
        assert (true_d <= want_d * (1 + 1e-5) + 1e-30).all()


@pytest.mark.parametrize("scale", [1e-12, 1e-6, 1e6, 1e12])
@pytest.mark.parametrize("k", [1, 20])
def test_route_extreme_magnitudes(scale, k):
    # the power-of-two operand scaling must keep small and large inputs inside fp16's range and the
    # returned distances inside the tolerance, which is relative to the norms
    rng = np.random.default_rng(int(abs(np.log10(scale))) + k)
    x = (rng.standard_normal((300, 64)) * scale).astype(np.float32)
    c = (rng.standard_normal((2500, 64)) * scale).astype(np.float32)
    ids, dists = (B.ivf_assign if k == 1 else lambda a, b: B.ivf_route(a, b, k))(_t(x), _t(c))
    B.ivf_check()
    parity.check_route(x, c, k, ids.cpu().numpy(), dists.cpu().numpy())


def test_route_mixed_magnitudes_between_points_and_centroids():
    # points much smaller than centroids and the other way round (the point scale is capped by the
    # centroid scale and floored 2^29 below it)
    rng = np.random.default_rng(77)
    for sx, sc in [(1e-4, 10.0), (300.0, 1e-2), (1.0, 1e5)]:
        x = (rng.standard_normal((200, 32)) * sx).astype(np.float32)
        c = (rng.standard_normal((1500, 32)) * sc).astype(np.float32)
        ids, dists = B.ivf_route(_t(x), _t(c), 12)
        B.ivf_check()
        parity.check_route(x, c, 12, ids.cpu().numpy(), dists.cpu().numpy())


@pytest.mark.parametrize("k", [1, 24])
def test_route_mixed_magnitudes_inside_one_table(k):
    # the operand scale is one power of two per matrix, so rows far below the matrix's largest
    # magnitude lose bits: the header promises the tolerance for pairs whose combined norm is at
    # least about 2^-9 of the largest centroid magnitude.  Here a tenth of the centroids and of the
    # points are 2^-4, 2^-6 or 2^-7 of the rest (small-small pairs sit at about 2^-5 of the maximum).
    rng = np.random.default_rng(91 + k)
    x = rng.standard_normal((400, 64)).astype(np.float32)
    c = rng.standard_normal((3000, 64)).astype(np.float32)
    for arr in (x, c):
        small = rng.choice(arr.shape[0], arr.shape[0] // 10, replace=False)
        arr[small] *= rng.choice([2.0 ** -4, 2.0 ** -6, 2.0 ** -7], small.size)[:, None].astype(np.float32)
    c[:40] = x[:40] * (1 + 1e-3)  # near neighbours, also among the small rows
    ids, dists = (B.ivf_assign if k == 1 else lambda a, b: B.ivf_route(a, b, k))(_t(x), _t(c))
    B.ivf_check()
    parity.check_route(x, c, k, ids.cpu().numpy(), dists.cpu().numpy())


@pytest.mark.parametrize("dtype,n,nlist,d,k", [
    ("u8", 2500, 4096, 32, 1), ("i8", 5000, 9000, 64, 1), ("u8", 1000, 40000, 16, 1),
    ("u8", 700, 4096, 128, 64), ("i8", 300, 1000, 100, 20),
])
def test_duplicate_centroids_lower_id_wins(dtype, n, nlist, d, k):
    """A third of the centroids are copies of other centroids, on integer data whose distances are
    exact: every tie between a centroid and its copy (in the same 8-column group, in another group of
    the same accumulator chunk, in another chunk, tile or CTA) must go to the lower id, as in the
    oracle's sort."""
    rng = np.random.default_rng(n + nlist + d + k)
    x = _points(rng, dtype, n, d, True)
    c = _centroids(rng, dtype, nlist, d, True)
    c[rng.integers(0, nlist, nlist // 3)] = c[rng.integers(0, nlist, nlist // 3)]
    if k == 1:
        ids, dists = B.ivf_assign(_t(x), _t(c))
    else:
        ids, dists = B.ivf_route(_t(x), _t(c), k)
    B.ivf_check()
    parity.check_route(x, c, k, ids.cpu().numpy(), dists.cpu().numpy(), exact=True)


@pytest.mark.parametrize("cluster,k", [(700, 64), (1500, 64), (3000, 128), (300, 20)])
def test_rows_with_many_times_the_usual_candidates(cluster, k):
    """A tight cluster of centroids sits next to some of the queries, at positions the threshold
    pass does not sample (it looks at every S-th centroid), so those rows' thresholds admit the whole
    cluster: several times the usual number of candidates reach the merge, which has to cut its
    buffer down in mid-gather (or hand the row to the general path) and still return the exact lists."""
    rng = np.random.default_rng(cluster + k)
    nlist, d, n = 32768, 32, 600
    c = (rng.standard_normal((nlist, d)) * 30 + 100).astype(np.float32)
    x = rng.integers(0, 256, (n, d)).astype(np.uint8)
    centre = x[0].astype(np.float32)
    stride = 64 if cluster <= nlist // 64 else 8
    where = np.flatnonzero(np.arange(nlist) % stride == 5)[:cluster]
    c[where] = centre + rng.standard_normal((where.size, d)).astype(np.float32) * 2.0
    x[:200] = np.clip(centre + rng.standard_normal((200, d)) * 3.0, 0, 255).astype(np.uint8)
    ids, dists = B.ivf_route(_t(x), _t(c), k)
    B.ivf_check()
    stats = parity.check_route(x, c, k, ids.cpu().numpy(), dists.cpu().numpy())
    assert stats["rows"] == n


def test_low_dimension_mixed_norms_order_within_tolerance():
    """d = 4, float rows, k = 256 of 1,000: centroid norms differ by an order of magnitude, so the
    tolerance differs from id to id; an id with a large norm may be ranked a few places off while the
    small-norm ids between keep their exact order (the case a random sweep found)."""
    rng = np.random.default_rng(770397)
    x = rng.standard_normal((5000, 4)).astype(np.float32)
    c = rng.standard_normal((1000, 4)).astype(np.float32)
    c[::7] *= 3.0
    ids, dists = B.ivf_route(_t(x), _t(c), 256)
    B.ivf_check()
    stats = parity.check_route(x, c, 256, ids.cpu().numpy(), dists.cpu().numpy())
    assert stats["max_err_over_tol"] <= 1.0
