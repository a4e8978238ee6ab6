"""Parity of the CUDA path (through the C-ABI) with the CPU oracle, element by element on the same
seeded inputs.  Distances within 1e-3 * (|x|^2 + |c|^2); id lists equal except inside that band;
integer-exact inputs bit for bit; counts bit-exact, sums within 1e-5 relative (exact for uint8)."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _route(x, c, k):
    if k == 1:
        ids, d = B.ivf_assign(_cuda(x), _cuda(c))
    else:
        ids, d = B.ivf_route(_cuda(x), _cuda(c), k)
    B.ivf_check()
    return ids.cpu().numpy(), d.cpu().numpy()


def _rand(n, nlist, d, dtype, seed):
    rng = np.random.default_rng(seed)
    if dtype == "u8":
        x = rng.integers(0, 256, (n, d)).astype(np.uint8)
        c = (rng.standard_normal((nlist, d)) * 40 + 100).astype(np.float32)
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
        c = rng.standard_normal((nlist, d)).astype(np.float32)
    return x, c


# several row tiles and centroid tiles, ragged tails on both, every supported K-slice count
SMALL = [
    (1, 1, 16, 1, "f32"), (1, 300, 128, 7, "f32"), (129, 257, 128, 1, "f32"), (300, 1000, 128, 1, "f32"),
    (300, 1000, 96, 1, "f32"), (1000, 5000, 128, 1, "u8"), (300, 1000, 128, 16, "f32"), (300, 3000, 96, 64, "f32"),
    (500, 20000, 128, 64, "u8"), (200, 700, 256, 8, "f32"), (200, 700, 192, 1, "u8"), (64, 40000, 16, 128, "f32"),
    (700, 513, 64, 512, "f32"), (130, 2000, 48, 2, "u8"), (40000, 3000, 128, 1, "u8"), (257, 9000, 96, 256, "f32"),
    (5, 600, 32, 600 - 88, "f32"),
    # long centroid sweeps per CTA: the sampled-threshold rule
    (128, 500000, 64, 64, "f32"), (100, 300000, 128, 40, "u8"), (128, 500000, 64, 17, "f32"), (300, 400000, 96, 128, "f32"),
]


@pytest.mark.parametrize("n,nlist,d,k,dtype", SMALL)
def test_small_cases_match_oracle(n, nlist, d, k, dtype):
    x, c = _rand(n, nlist, d, dtype, seed=n + nlist + d + k)
    ids, dists = _route(x, c, k)
    parity.check_route(x, c, k, ids, dists)


def test_k_equals_nlist_returns_sorted_permutation():
    x, c = _rand(50, 300, 64, "f32", 3)
    ids, dists = _route(x, c, 300)
    parity.check_route(x, c, 300, ids, dists)
    assert (np.sort(ids, 1) == np.arange(300)).all()


def test_config0_tiny_routing_full():
    cfg = synth.C0
    q, c = synth.routing_inputs(cfg)
    ids, dists = _route(q, c, cfg.nprobe)
    st = parity.check_route(q, c, cfg.nprobe, ids, dists)
    assert st["rows"] == cfg.nq


@pytest.mark.parametrize("n,nlist,d,k", [(300, 1500, 128, 1), (300, 1500, 128, 32), (260, 3000, 64, 100),
                                         (1000, 700, 16, 5), (200, 600, 256, 64)])
def test_integer_inputs_are_bit_exact_including_ties(n, nlist, d, k):
    # uint8 points and integer-valued centroids: every product and sum is exact in fp16 -> fp32 and in
    # fp64 alike, so ids (ties to the lower id) and distances must equal the oracle's bit for bit
    hi = 256 if d <= 128 else 128
    q, c = synth.integer_case(n, nlist, d, seed=d + k, hi=hi)
    if d == 16:
        q = (q % 4).astype(np.uint8)  # few distinct values: ties are plentiful
        c = np.floor(c / 64).astype(np.float32)
    ids, dists = _route(q, c, k)
    st = parity.check_route(q, c, k, ids, dists, exact=True)
    assert st["rows_identical"] == 1.0


@pytest.mark.parametrize("n,nlist,d,k,dtype", [(300, 5000, 128, 40, "u8"), (130, 2000, 96, 17, "f32"), (64, 70000, 64, 200, "f32")])
def test_brute_force_recomputation_of_failed_rows(n, nlist, d, k, dtype):
    # every row is declared failed by the merge, so all results come from the exact fallback kernel
    x, c = _rand(n, nlist, d, dtype, seed=7)
    B.ivf_debug_force_fallback(True)
    try:
        ids, dists = _route(x, c, k)
    finally:
        B.ivf_debug_force_fallback(False)
    parity.check_route(x, c, k, ids, dists)
    q, ci = synth.integer_case(200, 3000, 64, seed=3)
    B.ivf_debug_force_fallback(True)
    try:
        ids, dists = _route(q, ci, 50)
    finally:
        B.ivf_debug_force_fallback(False)
    parity.check_route(q, ci, 50, ids, dists, exact=True)


def test_brute_force_recomputation_with_ties_across_slices():
    # integer data (many equal distances), several centroid slices with a ragged last one, the
    # largest k: the (distance, id) order must survive both selection stages
    q, ci = synth.integer_case(40, 20000, 64, seed=5)
    B.ivf_debug_force_fallback(True)
    try:
        ids, dists = _route(q, ci, 512)
    finally:
        B.ivf_debug_force_fallback(False)
    parity.check_route(q, ci, 512, ids, dists, exact=True)


@pytest.mark.parametrize("k", [1, 8, 40])
def test_row_chunk_loop_of_large_calls(k):
    # big calls are split into row chunks that share the prepared centroids and the workspace;
    # force small chunks (ragged last one) and compare with the unsplit call and the oracle
    x, c = _rand(1000, 9000, 128, "u8", seed=31 + k)
    want = _route(x, c, k)
    B.ivf_debug_set_row_chunk(384)
    try:
        got = _route(x, c, k)
    finally:
        B.ivf_debug_set_row_chunk(0)
    assert (got[0] == want[0]).all() and (got[1] == want[1]).all()
    parity.check_route(x, c, k, got[0], got[1])


def test_sampled_threshold_rarely_needs_the_exact_recomputation():
    # the threshold pass lets about 4k candidates through; fewer than k should be a rare event
    q, c = synth.routing_inputs(synth.C1, nq=4096)
    B.ivf_debug_stats(True)
    ids, dists = _route(q, c, 64)
    st = B.ivf_debug_stats(False)
    assert st["fallback_rows"] <= 0.005 * 4096
    assert 64 <= st["log_entries"] / 4096 <= 6 * 64  # group records per row: near 4k, not the whole table
    rows = np.arange(0, 4096, 128)
    parity.check_route(q, c, 64, ids[rows], dists[rows], rows=rows)


@pytest.mark.parametrize("n,nlist,d,k,dtype", [(6200, 20000, 128, 40, "u8"), (7000, 70000, 96, 100, "f32"), (6145, 9000, 64, 17, "f32"),
                                               (20001, 20000, 64, 20, "u8")])  # the last: more row tiles than SMs
def test_threshold_pass_in_one_kernel_gives_the_same_results(n, nlist, d, k, dtype):
    # from 48 row tiles on, every CTA of the threshold pass takes whole row tiles across the entire
    # sample and finishes the thresholds itself; the split schedule (sketch kernel + merge launch)
    # computes the same statistic, so ids and distances must agree bit for bit
    x, c = _rand(n, nlist, d, dtype, seed=n)
    ids, dists = _route(x, c, k)
    B.ivf_debug_set_threshold_pass(True)
    try:
        ids2, dists2 = _route(x, c, k)
    finally:
        B.ivf_debug_set_threshold_pass(False)
    assert (ids == ids2).all() and (dists == dists2).all()
    rows = np.arange(0, n, 37)
    parity.check_route(x, c, k, ids[rows], dists[rows], rows=rows)


@pytest.mark.parametrize("n", [1, 3, 8, 9, 16, 17, 32, 33])  # main pass: up to 16 rows, up to 32 against the largest table
@pytest.mark.parametrize("nlist,d,k,dtype", [(300000, 128, 64, "u8"), (90000, 96, 128, "f32"), (33000, 64, 17, "f32")])
def test_thresholds_finished_by_the_main_pass_give_the_same_results(n, nlist, d, k, dtype):
    # batches of at most 16 rows (32 when every CTA has tiles enough to compute meanwhile): the epilogue
    # warps of the main pass merge the partial sketches of the threshold pass themselves (a warp per
    # row, four rows per warp at most); the merge kernel computes the same order
    # statistic, so the two schedules must agree bit for bit -- with one or several sketches per lane
    x, c = _rand(n, nlist, d, dtype, seed=n + nlist)
    ids, dists = _route(x, c, k)
    B.ivf_debug_set_threshold_pass(True)
    try:
        ids2, dists2 = _route(x, c, k)
    finally:
        B.ivf_debug_set_threshold_pass(False)
    assert (ids == ids2).all() and (dists == dists2).all()
    parity.check_route(x, c, k, ids, dists)


def test_duplicate_centroids_resolve_to_lower_id():
    _, c = _rand(1, 700, 128, "f32", 9)
    c[500] = c[20]
    c[699] = c[20]
    ids, dists = _route(c[[20, 500, 699, 3]], c, 4)
    assert ids[0, :3].tolist() == [20, 500, 699] and ids[1, :3].tolist() == [20, 500, 699]
    assert ids[3, 0] == 3 and (dists[:, 0] <= 1e-3 * 2 * (c[20] ** 2).sum()).all()


def test_scaling_of_tiny_and_huge_magnitudes():
    x, c = _rand(200, 900, 96, "f32", 4)
    for s in (1e-6, 3e4):
        ids, dists = _route((x * s).astype(np.float32), (c * s).astype(np.float32), 10)
        parity.check_route((x * s).astype(np.float32), (c * s).astype(np.float32), 10, ids, dists)


def test_run_to_run_determinism():
    x, c = _rand(700, 6000, 128, "u8", 5)
    a = _route(x, c, 40)
    for _ in range(2):
        b = _route(x, c, 40)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


@pytest.mark.parametrize("n,nlist,d,k,dtype", [(8, 30000, 128, 64, "u8"), (300, 5000, 96, 10, "f32"), (2048, 9000, 128, 1, "u8")])
def test_prepared_centroids_give_identical_results(n, nlist, d, k, dtype):
    x, c = _rand(n, nlist, d, dtype, seed=n + k)
    h = B.PreparedCentroids(_cuda(c))
    for rep in range(2):  # the handle is reused across batches
        xs = x if rep == 0 else np.ascontiguousarray(x[::-1])
        ids_p, d_p = B.ivf_route_prepared(h, _cuda(xs), k)
        B.ivf_check()
        ids, dists = B.ivf_route(_cuda(xs), _cuda(c), k)
        B.ivf_check()
        assert (ids_p == ids).all() and (d_p == dists).all()
        parity.check_route(xs, c, k, ids_p.cpu().numpy(), d_p.cpu().numpy())
    h.close()


def test_no_distances_requested():
    x, c = _rand(200, 500, 64, "f32", 6)
    ids, none = B.ivf_route(_cuda(x), _cuda(c), 5, want_dists=False)
    B.ivf_check()
    assert none is None
    ids2, _ = _route(x, c, 5)
    assert (ids.cpu().numpy() == ids2).all()


# ---------------------------------------------------------------- full-size configurations
def _full_size(cfg, sample, stats=False):
    """The whole configuration through the C-ABI in its production launch shape; the full oracle on
    `sample` rows spread evenly over the batch (so every row chunk of a chunked call is hit) plus a
    seeded random draw, and the definition re-checked for every returned (row, id) pair."""
    q, c = synth.routing_inputs(cfg)
    if stats:
        B.ivf_debug_stats(True)
    ids, dists = _route(q, c, cfg.nprobe)
    st = B.ivf_debug_stats(False) if stats else None
    even = np.unique(np.linspace(0, cfg.nq - 1, sample // 2).astype(np.int64))
    rest = np.setdiff1d(np.arange(cfg.nq), even)
    rnd = np.random.default_rng(cfg.index).choice(rest, sample - even.size, replace=False)
    rows = np.sort(np.concatenate([even, rnd]))
    res = parity.check_route(q, c, cfg.nprobe, ids[rows], dists[rows], rows=rows)
    parity.check_all_row_distances(q, c, cfg.nprobe, ids, dists)
    return res, st, (q, c, ids, dists)


def test_config1_sift_shaped_full_size():
    res, _, _ = _full_size(synth.C1, 2048)
    assert res["rows"] == 2048


def test_config2_deep_shaped_full_size():
    res, _, _ = _full_size(synth.C2, 1024)
    assert res["rows"] == 1024


def test_config4_stress_full_size():
    # 11 row chunks; 2,048 oracle rows spread over all of them
    res, st, _ = _full_size(synth.C4, 2048, stats=True)
    assert res["rows"] == 2048
    assert st["fallback_rows"] <= 0.001 * synth.C4.nq


def test_config4_shape_rows_through_the_exact_recomputation():
    # the recomputation path at the C4 table size (128 centroid slices per row): a C4-shaped subset
    # of rows is forced through it and must agree with the oracle like any other result
    cfg = synth.C4
    q, c = synth.routing_inputs(cfg)
    sub = np.ascontiguousarray(q[np.random.default_rng(44).choice(cfg.nq, 48, replace=False)])
    B.ivf_debug_stats(True)
    B.ivf_debug_force_fallback(True)
    try:
        ids, dists = _route(sub, c, cfg.nprobe)
    finally:
        B.ivf_debug_force_fallback(False)
    st = B.ivf_debug_stats(False)
    assert st["fallback_rows"] == 48
    parity.check_route(sub, c, cfg.nprobe, ids, dists)
    # the regular path sums the same fp16 products in another order, so its lists may differ from the
    # recomputed ones where keys are nearly equal -- both must satisfy the rule, and share nearly all ids
    ids2, dists2 = _route(sub, c, cfg.nprobe)
    parity.check_route(sub, c, cfg.nprobe, ids2, dists2)
    shared = np.mean([np.intersect1d(a, b).size for a, b in zip(ids, ids2)]) / cfg.nprobe
    assert shared > 0.98


def test_config3_chunk_assignment_full_width_sampled():
    x = synth.sift_like_rows(0)
    c = synth.sift_like_centroids(synth.C3_NLIST)
    ids, dists = _route(x, c, 1)
    rows = np.random.default_rng(3).choice(x.shape[0], 96, replace=False)
    parity.check_route(x, c, 1, ids[rows], dists[rows], rows=rows)
    # every returned distance re-checked against the definition (n*d work)
    D = oracle.pair_dists(x, c, np.arange(x.shape[0]), ids)
    tol = 1e-3 * (oracle.sqnorms(x) + oracle.sqnorms(c)[ids])
    assert (np.abs(dists - D) <= tol).all()


# ---------------------------------------------------------------- Lloyd update
@pytest.mark.parametrize("dtype,n,nlist,d", [("u8", 5000, 300, 128), ("f32", 5000, 300, 96), ("u8", 70000, 65536, 128),
                                             ("f32", 3000, 7, 256), ("u8", 1, 5, 16), ("f32", 9000, 4097, 32)])
def test_update_matches_oracle_and_accumulates(dtype, n, nlist, d):
    rng = np.random.default_rng(n + nlist)
    x = rng.integers(0, 256, (n, d)).astype(np.uint8) if dtype == "u8" else rng.standard_normal((n, d)).astype(np.float32)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    if nlist > 10:
        ids[ids == 3] = 4  # an empty list
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    xt, it = _cuda(x), _cuda(ids)
    h = n // 2
    B.ivf_centroid_update(xt[:h].contiguous(), it[:h].contiguous(), sums, counts) if h else None
    B.ivf_centroid_update(xt[h:].contiguous(), it[h:].contiguous(), sums, counts)
    B.ivf_check()
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy())
    assert counts.sum().item() == n


def test_update_flags_and_skips_bad_ids():
    x = np.arange(4 * 16, dtype=np.float32).reshape(4, 16)
    ids = np.array([1, 9, -1, 0], np.int32)
    sums = torch.zeros((3, 16), dtype=torch.float32, device="cuda")
    counts = torch.zeros((3,), dtype=torch.int64, device="cuda")
    B.ivf_centroid_update(_cuda(x), _cuda(ids), sums, counts)
    with pytest.raises(B.IvfError) as e:
        B.ivf_check()
    assert e.value.code == B.IVF_ERR_BAD_ID
    assert counts.cpu().tolist() == [1, 1, 0]
    assert (sums.cpu().numpy()[1] == x[0]).all() and (sums.cpu().numpy()[0] == x[3]).all()
    B.ivf_check()  # the status word was cleared


def test_update_run_to_run_reproducibility():
    # byte rows: sums and counts bit-identical over three runs; float rows: counts identical, sums
    # within the rounding of a different summation order
    rng = np.random.default_rng(12)
    n, nlist, d = 60000, 900, 64
    ids = _cuda(rng.integers(0, nlist, n).astype(np.int32))
    for dtype in ("u8", "f32"):
        x = rng.integers(0, 256, (n, d)).astype(np.uint8) if dtype == "u8" else rng.standard_normal((n, d)).astype(np.float32)
        xt = _cuda(x)
        runs = []
        for _ in range(3):
            sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
            counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
            B.ivf_centroid_update(xt, ids, sums, counts)
            B.ivf_check()
            runs.append((sums.cpu().numpy(), counts.cpu().numpy()))
        for s, c in runs[1:]:
            assert (c == runs[0][1]).all()
            if dtype == "u8":
                assert (s == runs[0][0]).all()
            else:
                mag = np.zeros((nlist, d))
                np.add.at(mag, ids.cpu().numpy(), np.abs(x.astype(np.float64)))
                assert (np.abs(s.astype(np.float64) - runs[0][0]) <= 1e-5 * mag + 1e-30).all()


def test_finalize_matches_oracle_and_keeps_empty_lists():
    rng = np.random.default_rng(1)
    sums = rng.standard_normal((50, 32)).astype(np.float32) * 100
    counts = rng.integers(0, 5, 50).astype(np.int64)
    old = rng.standard_normal((50, 32)).astype(np.float32)
    ct = _cuda(old.copy())
    B.ivf_centroid_finalize(_cuda(sums), _cuda(counts), ct)
    want = oracle.finalize(sums.astype(np.float64), counts, old)
    got = ct.cpu().numpy()
    assert (got[counts == 0] == old[counts == 0]).all()
    np.testing.assert_allclose(got, want, rtol=2e-7)  # fp32 divide vs fp64 divide then rounding: <= 1 ulp


# ---------------------------------------------------------------- cluster-major reorder
@pytest.mark.parametrize("dtype,n,nlist,d", [("u8", 20000, 700, 128), ("f32", 5000, 4097, 96), ("u8", 300, 5, 16),
                                             ("f32", 1, 3, 32)])
def test_cluster_major_reorder(dtype, n, nlist, d):
    rng = np.random.default_rng(n)
    x = rng.integers(0, 256, (n, d)).astype(np.uint8) if dtype == "u8" else rng.standard_normal((n, d)).astype(np.float32)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    if nlist > 10:
        ids[ids == 2] = 3  # an empty list
    out, offsets, order = B.ivf_cluster_major_reorder(_cuda(x), _cuda(ids), nlist)
    B.ivf_check()
    out, offsets, order = out.cpu().numpy(), offsets.cpu().numpy(), order.cpu().numpy()
    o_off, o_order = oracle.reorder(ids, nlist)
    assert (offsets == o_off).all()                       # unique: where every list starts and ends
    assert (np.sort(order) == np.arange(n)).all()         # a permutation of the rows
    assert (ids[order] == np.repeat(np.arange(nlist), np.diff(o_off))).all()  # list-major
    for l in (0, nlist // 2, nlist - 1):                  # inside a list any order is valid: compare the sets
        assert sorted(order[o_off[l]:o_off[l + 1]].tolist()) == o_order[o_off[l]:o_off[l + 1]].tolist()
    assert (out == x[order]).all()


@pytest.mark.parametrize("dtype,d", [("u8", 128), ("f32", 36)])
def test_cluster_major_reorder_drops_rows_with_bad_ids(dtype, d):
    # rows whose id is outside [0, nlist) are left out: the kept rows fill the front of the layout, the
    # positions after them read order = -1 and a zero row, and the status word reports the bad ids
    n, nlist = 5000, 300
    rng = np.random.default_rng(17)
    x = rng.integers(1, 256, (n, d)).astype(np.uint8) if dtype == "u8" else (rng.standard_normal((n, d)).astype(np.float32) + 5)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    bad = rng.choice(n, 37, replace=False)
    ids[bad[:20]] = -1 - rng.integers(0, 1000, 20).astype(np.int32)
    ids[bad[20:]] = nlist + rng.integers(0, 1000, 17).astype(np.int32)
    out, offsets, order = B.ivf_cluster_major_reorder(_cuda(x), _cuda(ids), nlist)
    with pytest.raises(B.IvfError) as e:
        B.ivf_check()
    assert e.value.code == B.IVF_ERR_BAD_ID
    out, offsets, order = out.cpu().numpy(), offsets.cpu().numpy(), order.cpu().numpy()
    good = np.flatnonzero((ids >= 0) & (ids < nlist))
    o_off, _ = oracle.reorder(ids[good], nlist)
    kept = n - 37
    assert (offsets == o_off).all() and offsets[-1] == kept
    assert (np.sort(order[:kept]) == good).all()
    assert (ids[order[:kept]] == np.repeat(np.arange(nlist), np.diff(o_off))).all()
    assert (out[:kept] == x[order[:kept]]).all()
    assert (order[kept:] == -1).all() and (out[kept:] == 0).all()
    B.ivf_check()


# ---------------------------------------------------------------- host streaming
def test_route_from_pinned_host_memory():
    x, c = _rand(3000, 2000, 128, "u8", 12)
    xt = torch.from_numpy(x).pin_memory()
    ids, dists = B.ivf_route(xt, _cuda(c), 8)
    B.ivf_check()
    ids2, d2 = _route(x, c, 8)
    assert (ids.cpu().numpy() == ids2).all() and (dists.cpu().numpy() == d2).all()


@pytest.mark.parametrize("host", [True, False])
def test_assign_update_streamed_in_chunks(host):
    n, nlist, d = 10500, 400, 128
    x = synth.sift_like_rows(7, rows=n)
    c = synth.sift_like_centroids(nlist)
    xt = torch.from_numpy(x).pin_memory() if host else _cuda(x)
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    ids = torch.empty((n,), dtype=torch.int32, device="cuda")
    dists = torch.empty((n,), dtype=torch.float32, device="cuda")
    B.ivf_assign_update(xt, _cuda(c), sums, counts, ids, dists, chunk_rows=2048)  # 6 chunks, ragged tail
    B.ivf_check()
    parity.check_route(x, c, 1, ids.cpu().numpy(), dists.cpu().numpy())
    parity.check_update(x, ids.cpu().numpy(), nlist, sums.cpu().numpy(), counts.cpu().numpy())
    # without id output
    sums2, counts2 = torch.zeros_like(sums), torch.zeros_like(counts)
    B.ivf_assign_update(xt, _cuda(c), sums2, counts2, chunk_rows=4096)
    B.ivf_check()
    assert (counts2 == counts).all() and (sums2 == sums).all()


def _pinned(shape, dtype, fill):
    t = torch.full(shape, fill, dtype=dtype).pin_memory()
    return t


@pytest.mark.parametrize("host_in", [False, True])
@pytest.mark.parametrize("k,with_dists", [(1, True), (8, True), (40, False)])
def test_results_in_pinned_host_memory(host_in, k, with_dists):
    # the kernels write to staging buffers of the workspace; every row chunk is read back on the
    # library's own stream and the caller's stream waits for the last copy before the call counts as done
    n, nlist, d = 7000, 3000, 64
    x, c = _rand(n, nlist, d, "f32", 77)
    want_ids, want_d = _route(x, c, k)
    xt = torch.from_numpy(x).pin_memory() if host_in else _cuda(x)
    shape = (n,) if k == 1 else (n, k)
    ids_h = _pinned(shape, torch.int32, -7)
    d_h = _pinned(shape, torch.float32, -7.0) if with_dists else None
    B.ivf_debug_set_row_chunk(1536)  # five chunks with a ragged tail: both staging pairs are reused
    try:
        if k == 1:
            B.ivf_assign(xt, _cuda(c), ids_h, d_h, want_dists=with_dists)
        else:
            B.ivf_route(xt, _cuda(c), k, ids_h, d_h, want_dists=with_dists)
        torch.cuda.current_stream().synchronize()  # no ivf_check here: the stream alone must cover the read-back
    finally:
        B.ivf_debug_set_row_chunk(0)
    assert (ids_h.numpy() == want_ids).all()
    if with_dists:
        assert (d_h.numpy() == want_d).all()
    B.ivf_check()


def test_prepared_table_with_results_in_host_memory():
    x, c = _rand(900, 40000, 128, "u8", 31)
    want_ids, want_d = _route(x, c, 64)
    h = B.PreparedCentroids(_cuda(c))
    try:
        ids_h, d_h = _pinned((900, 64), torch.int32, -1), _pinned((900, 64), torch.float32, -1.0)
        xt = torch.from_numpy(x).pin_memory()  # alive until the copy has run
        B.ivf_route_prepared(h, xt, 64, ids_h, d_h)
        torch.cuda.current_stream().synchronize()
        assert (ids_h.numpy() == want_ids).all() and (d_h.numpy() == want_d).all()
        B.ivf_check()
    finally:
        h.close()


def test_deferred_read_back_of_host_results():
    # serving loop: with deferred read-back the calls do not wait for their copies; two staging pairs
    # are used in turn, so a third call must wait for the first one's copy before it reuses the pair
    n, nlist, d, k = 4000, 5000, 128, 32
    c = _cuda(_rand(1, nlist, d, "u8", 5)[1])
    batches = [_rand(n, nlist, d, "u8", 100 + i)[0] for i in range(5)]
    want = []
    for xb in batches:
        ids, dd = B.ivf_route(_cuda(xb), c, k)
        want.append((ids.cpu().numpy(), dd.cpu().numpy()))
    hosts = [(_pinned((n, k), torch.int32, -1), _pinned((n, k), torch.float32, -1.0)) for _ in batches]
    pinned_in = [torch.from_numpy(xb).pin_memory() for xb in batches]  # alive until the copies have run
    B.ivf_set_deferred_host_outputs(True)
    try:
        for xt, (ih, dh) in zip(pinned_in, hosts):
            B.ivf_route(xt, c, k, ih, dh)
        B.ivf_wait_host_outputs()
        torch.cuda.current_stream().synchronize()
        for (wi, wd), (ih, dh) in zip(want, hosts):
            assert (ih.numpy() == wi).all() and (dh.numpy() == wd).all()
        # ivf_check alone waits for outstanding read-backs as well
        ih, dh = _pinned((n, k), torch.int32, -1), _pinned((n, k), torch.float32, -1.0)
        B.ivf_route(_cuda(batches[0]), c, k, ih, dh)
        B.ivf_check()
        assert (ih.numpy() == want[0][0]).all() and (dh.numpy() == want[0][1]).all()
    finally:
        B.ivf_set_deferred_host_outputs(False)


def test_assign_update_with_ids_in_host_memory():
    n, nlist, d = 9000, 300, 128
    x = synth.sift_like_rows(3, rows=n)
    c = synth.sift_like_centroids(nlist)
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    ids_h = _pinned((n,), torch.int32, -1)
    xt = torch.from_numpy(x).pin_memory()  # alive until the copies have run
    B.ivf_assign_update(xt, _cuda(c), sums, counts, ids_h, None, chunk_rows=2048)
    torch.cuda.current_stream().synchronize()
    ids = ids_h.numpy().copy()
    B.ivf_check()
    want, _ = _route(x, c, 1)
    assert (ids == want).all()
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy())


def test_mixed_host_and_device_outputs_are_rejected():
    x, c = _rand(100, 200, 64, "f32", 1)
    ids_h = _pinned((100, 4), torch.int32, 0)
    d_dev = torch.empty((100, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(B.IvfError) as e:
        B.ivf_route(_cuda(x), _cuda(c), 4, ids_h, d_dev)
    assert e.value.code == B.IVF_ERR_INVALID_ARG
    ids_dev = torch.empty((100, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(B.IvfError):
        B.ivf_route(_cuda(x), _cuda(c), 4, ids_dev, _pinned((100, 4), torch.float32, 0.0))


def test_pageable_host_memory_is_rejected():
    x, c = _rand(100, 200, 64, "f32", 1)
    xt = torch.from_numpy(x)
    with pytest.raises((ValueError, B.IvfError)):
        B.ivf_route(xt, _cuda(c), 4)
    buf = np.zeros((100, 64), np.float32)
    ids = torch.empty((100, 4), dtype=torch.int32, device="cuda")
    rc = B.lib().ivf_route(buf.ctypes.data, 100, 64, 0, _cuda(c).data_ptr(), 200, 4, ids.data_ptr(), None, None)
    assert rc in (B.IVF_ERR_INVALID_ARG, B.IVF_ERR_CUDA)


# ---------------------------------------------------------------- Lloyd iterations, step-wise against the oracle
def test_lloyd_twin_stepwise():
    n, nlist, d, iters = 20000, 512, 128, 3
    x = synth.sift_like_rows(1, rows=n)
    init = x[synth.init_sample(n, nlist)].astype(np.float32)
    xt = _cuda(x)
    ct = _cuda(init.copy())
    inertia = []
    for _ in range(iters):
        c_now = ct.cpu().numpy().copy()
        sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
        counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
        ids = torch.empty((n,), dtype=torch.int32, device="cuda")
        dists = torch.empty((n,), dtype=torch.float32, device="cuda")
        B.ivf_assign_update(xt, ct, sums, counts, ids, dists, chunk_rows=8192)
        B.ivf_centroid_finalize(sums, counts, ct)
        B.ivf_check()
        g_ids = ids.cpu().numpy()
        # the oracle is fed the GPU's current centroids, so a tolerated near-tie cannot compound
        parity.check_route(x, c_now, 1, g_ids, dists.cpu().numpy())
        parity.check_update(x, g_ids, nlist, sums.cpu().numpy(), counts.cpu().numpy())
        want = oracle.finalize(sums.cpu().numpy().astype(np.float64), counts.cpu().numpy(), c_now)
        np.testing.assert_allclose(ct.cpu().numpy(), want, rtol=2e-7)
        inertia.append(float(dists.double().sum().item()))
    assert all(b <= a * (1 + 1e-6) for a, b in zip(inertia, inertia[1:]))
    _, _, o_inertia = oracle.lloyd(x, init, iters)
    np.testing.assert_allclose(inertia, o_inertia, rtol=1e-3)


# ---------------------------------------------------------------- bounded waits
def test_expired_wait_is_reported_and_context_survives():
    # a wait on a barrier that nothing completes runs out after the (shortened) limit; the kernel
    # returns normally, the host reads the status, and the same context keeps computing correctly
    x, c = _rand(300, 1000, 128, "f32", 2)
    B.ivf_debug_set_wait_limit_ns(2_000_000)  # 2 ms
    try:
        B.ivf_debug_wait_probe()
        with pytest.raises(B.IvfError) as e:
            B.ivf_check()
        assert e.value.code == B.IVF_ERR_DEVICE_TIMEOUT and "99" in str(e.value)
    finally:
        B.ivf_debug_set_wait_limit_ns(0)
    B.ivf_check()
    ids, dists = _route(x, c, 1)
    parity.check_route(x, c, 1, ids, dists)


@pytest.mark.parametrize("dtype,n,nlist,d", [("u8", 300000, 3, 128), ("f32", 200000, 1, 96), ("u8", 1 << 20, 256, 4),
                                              ("f32", 500000, 17, 36), ("u8", 70000, 16, 256)])
def test_update_with_few_long_lists(dtype, n, nlist, d):
    # lists of thousands of members are cut into pieces (one warp each) whose partial sums are added
    # in piece order; uint8 sums stay exact, float sums inside the tolerance, counts exact; the sums
    # accumulate on top of what is there
    rng = np.random.default_rng(n % 1000 + nlist)
    if dtype == "u8":
        x = rng.integers(0, 16, (n, d)).astype(np.uint8)  # small values: list sums stay below 2^24
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    ids[: n // 3] = 0  # one list much longer than the others
    base = rng.integers(0, 9, (nlist, d)).astype(np.float32)
    sums = torch.from_numpy(base.copy()).cuda()
    counts = torch.full((nlist,), 5, dtype=torch.int64, device="cuda")
    B.ivf_centroid_update(_cuda(x), _cuda(ids), sums, counts)
    B.ivf_check()
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy(), base.astype(np.float64), np.full(nlist, 5, np.int64))
