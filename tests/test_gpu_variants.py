"""GPU parity of the input variants: signed bytes and row lengths that are a multiple of 4 but not
of 16 (SPACEV-shaped data is int8 with d = 100, Table 2), through every entry point that takes
points: routing, assignment, centroid update, list-major reorder, candidate assignment and the
residual-PQ chain."""
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


def _route(x, c, k):
    if k == 1:
        ids, d = B.ivf_assign(_t(x), _t(c))
    else:
        ids, d = B.ivf_route(_t(x), _t(c), k)
    B.ivf_check()
    return ids.cpu().numpy(), d.cpu().numpy()


def _case(dtype, n, nlist, d, seed):
    rng = np.random.default_rng(seed)
    if dtype == "i8":
        x, c = synth.spacev_like(n, nlist, seed, d)
    elif dtype == "u8":
        x = rng.integers(0, 256, (n, d)).astype(np.uint8)
        c = (rng.standard_normal((nlist, d)) * 40 + 100).astype(np.float32)
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
        c = rng.standard_normal((nlist, d)).astype(np.float32)
    return x, c


@pytest.mark.parametrize("dtype,n,nlist,d,k", [
    ("i8", 700, 3000, 100, 1), ("i8", 700, 3000, 100, 32), ("i8", 300, 20000, 100, 64), ("i8", 500, 2000, 128, 8),
    ("u8", 400, 2500, 100, 16), ("u8", 333, 900, 20, 1), ("f32", 400, 2500, 100, 16), ("f32", 257, 1000, 4, 3),
    ("f32", 300, 1500, 36, 1), ("i8", 200, 400000, 100, 40), ("f32", 129, 700, 252, 5),
])
def test_route_and_assign_match_oracle(dtype, n, nlist, d, k):
    x, c = _case(dtype, n, nlist, d, seed=n + d + k)
    ids, dists = _route(x, c, k)
    parity.check_route(x, c, k, ids, dists)


def test_signed_integer_inputs_are_bit_identical():
    # int8 points and integer centroids: all arithmetic exact, ties plentiful
    rng = np.random.default_rng(12)
    x = rng.integers(-128, 128, (300, 100)).astype(np.int8)
    c = rng.integers(-128, 128, (2000, 100)).astype(np.float32)
    ids, dists = _route(x, c, 24)
    st = parity.check_route(x, c, 24, ids, dists, exact=True)
    assert st["rows_identical"] == 1.0
    x2 = (rng.integers(-2, 3, (200, 100))).astype(np.int8)
    c2 = (rng.integers(-2, 3, (900, 100))).astype(np.float32)
    ids, dists = _route(x2, c2, 10)
    st = parity.check_route(x2, c2, 10, ids, dists, exact=True)
    assert st["rows_identical"] == 1.0


@pytest.mark.parametrize("dtype,d", [("i8", 100), ("i8", 128), ("u8", 100), ("f32", 100)])
def test_update_reorder_and_lloyd_step(dtype, d):
    n, nlist = 5000, 300
    x, c = _case(dtype, n, nlist, d, seed=d)
    ids = np.random.default_rng(d).integers(0, nlist, n).astype(np.int32)
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    B.ivf_centroid_update(_t(x), _t(ids), sums, counts)
    B.ivf_check()
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy())
    xr, offsets, order = B.ivf_cluster_major_reorder(_t(x), _t(ids), nlist)
    B.ivf_check()
    want_off, _ = O.reorder(ids, nlist)
    assert (offsets.cpu().numpy() == want_off).all()
    order = order.cpu().numpy()
    assert (np.sort(order) == np.arange(n)).all() and (np.diff(ids[order]) >= 0).all()
    assert (xr.cpu().numpy() == x[order]).all()
    # one streamed assign + update pass against the oracle fed with the GPU's ids
    sums.zero_(); counts.zero_()
    a_ids = torch.empty((n,), dtype=torch.int32, device="cuda")
    a_d = torch.empty((n,), dtype=torch.float32, device="cuda")
    B.ivf_assign_update(_t(x), _t(c), sums, counts, a_ids, a_d, chunk_rows=1536)
    B.ivf_check()
    g = a_ids.cpu().numpy()
    parity.check_route(x, c, 1, g, a_d.cpu().numpy())
    parity.check_update(x, g, nlist, sums.cpu().numpy(), counts.cpu().numpy())


def test_host_resident_int8_chunks():
    x, c = synth.spacev_like(3000, 500, seed=4)
    xh = torch.from_numpy(x).pin_memory()
    ids, d = B.ivf_assign(xh, _t(c))
    B.ivf_check()
    parity.check_route(x, c, 1, ids.cpu().numpy(), d.cpu().numpy())


def test_candidates_and_pq_with_signed_bytes():
    n, nlist, d, pq_m = 3000, 40, 100, 20
    x, c = synth.spacev_like(n, nlist, seed=5)
    ids, offsets = synth.skewed_list_ids(n, nlist, seed=5)
    cand = np.random.default_rng(5).integers(0, nlist, (n, 8)).astype(np.int32)
    g_ids, g_d = B.ivf_assign_candidates(_t(x), _t(c), _t(cand))
    B.ivf_check()
    w_ids, w_d = O.assign_candidates(x, c, cand)
    assert (g_ids.cpu().numpy() == w_ids).mean() > 0.999
    assert np.allclose(g_d.cpu().numpy(), O.pair_dists(x, c, np.arange(n), g_ids.cpu().numpy()), rtol=1e-5)
    cb = synth.pq_codebooks(pq_m, d // pq_m, 12.0, seed=5)
    want_codes = O.pq_encode(x, ids, c, cb)
    got_codes = B.ivf_pq_encode(_t(x), _t(ids), _t(c), _t(cb))
    B.ivf_check()
    assert (got_codes.cpu().numpy() == want_codes).all()
    q = x[:11]
    probes = synth.distinct_probes(11, nlist, 6, seed=5)
    want = O.pq_search(q, c, probes, offsets, want_codes, cb, 100)
    got = B.ivf_pq_search(_t(q), _t(c), _t(probes), _t(offsets), _t(want_codes), _t(cb), 100)
    B.ivf_check()
    assert (got[0].cpu().numpy() == want[0]).all() and (got[2].cpu().numpy() == want[2]).all()
    assert (got[1].cpu().numpy().view(np.uint32) == want[1].view(np.uint32)).all()


@pytest.mark.parametrize("nq,nlist,k", [(8, 40000, 64), (700, 9000, 1), (300, 3000, 12)])
def test_calls_can_be_captured_in_a_cuda_graph(nq, nlist, k):
    """Once the workspace has been sized by a first call of the same shape, a call enqueues only
    kernels and memsets, so a caller may capture it in a CUDA graph; the replay must give the
    results of the plain call (and those match the oracle)."""
    rng = np.random.default_rng(nq + nlist)
    x = rng.integers(0, 256, (nq, 64)).astype(np.uint8)
    c = (rng.standard_normal((nlist, 64)) * 30 + 110).astype(np.float32)
    xt, ct = _t(x), _t(c)
    h = B.PreparedCentroids(ct)
    ids = torch.empty((nq, k), dtype=torch.int32, device="cuda")
    ds = torch.empty((nq, k), dtype=torch.float32, device="cuda")

    def call():
        if k == 1:
            B.ivf_assign(xt, ct, ids.view(-1), ds.view(-1))
        else:
            B.ivf_route_prepared(h, xt, k, ids, ds)

    call()
    B.ivf_check()
    want_ids, want_d = ids.clone(), ds.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        call()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            call()
    for _ in range(3):
        ids.zero_()
        ds.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(ids, want_ids) and torch.equal(ds, want_d)
    B.ivf_check()
    parity.check_route(x, c, k, ids.cpu().numpy(), ds.cpu().numpy())
    h.close()
