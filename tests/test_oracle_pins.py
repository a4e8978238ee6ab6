"""Pins for the CPU oracle: every function of oracle/ is checked against something other than
itself: hand-computed values, closed forms, library routines, brute force and invariants."""
import itertools
import json
import os

import numpy as np
import pytest
import scipy.spatial.distance as ssd

from oracle import oracle
from paper_2608_08751_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")


def _golden():
    with open(GOLDEN) as f:
        return json.load(f)


# ---------------------------------------------------------------- hand-computed values
@pytest.mark.parametrize("case", _golden()["route"], ids=lambda c: c["cite"][:30])
def test_hand_cases_route(case):
    dt = np.uint8 if case["dtype"] == "u8" else np.float32
    q = np.array(case["queries"], dt)
    c = np.array(case["centroids"], np.float32)
    ids, dists, nxt = oracle.route(q, c, case["k"])
    assert ids.tolist() == case["ids"]
    assert dists.tolist() == [[float(v) for v in row] for row in case["dists"]]
    if "next" in case:
        assert nxt.tolist() == [float(v) for v in case["next"]]
    else:
        assert np.isinf(nxt).all()  # k == nlist


def test_hand_case_lloyd():
    g = _golden()["lloyd"]
    x = np.array(g["points"], np.float32)
    init = x[np.array(g["init_rows"])]
    c, ids, inertia = oracle.lloyd(x, init, g["iters"])
    assert ids.tolist() == g["ids"]
    np.testing.assert_allclose(inertia, g["inertia"], rtol=1e-6)
    np.testing.assert_allclose(c, g["centroids"], rtol=1e-6)


# ---------------------------------------------------------------- closed forms
def test_one_hot_closed_form():
    # x = a e_p, c = b e_q  ->  (a-b)^2 if p == q else a^2 + b^2
    d = 7
    a = np.array([3.0, -2.0, 0.5, 4.0], np.float32)
    p = np.array([0, 3, 6, 3])
    b = np.array([1.0, 5.0, -1.5], np.float32)
    qd = np.array([3, 0, 6])
    x = np.zeros((4, d), np.float32); x[np.arange(4), p] = a
    c = np.zeros((3, d), np.float32); c[np.arange(3), qd] = b
    ids, dists, _ = oracle.route(x, c, 3)
    for i in range(4):
        for pos in range(3):
            j = ids[i, pos]
            want = (a[i] - b[j]) ** 2 if p[i] == qd[j] else a[i] ** 2 + b[j] ** 2
            assert dists[i, pos] == pytest.approx(float(want), rel=1e-12)
        assert sorted(ids[i].tolist()) == [0, 1, 2]


def test_unit_norm_identity():
    # unit vectors in the plane: |x-c|^2 = 2 - 2 cos(angle between them), within [0, 4]
    ang_x = np.array([0.0, 0.3, 2.0, 3.1])
    ang_c = np.array([0.1, 1.0, 2.5, -3.0, 0.3])
    x = np.stack([np.cos(ang_x), np.sin(ang_x)], 1).astype(np.float32)
    c = np.stack([np.cos(ang_c), np.sin(ang_c)], 1).astype(np.float32)
    ids, dists, _ = oracle.route(x, c, 5)
    for i in range(4):
        for pos in range(5):
            want = 2 - 2 * np.cos(ang_x[i] - ang_c[ids[i, pos]])
            assert dists[i, pos] == pytest.approx(want, abs=2e-6)  # inputs were rounded to fp32
    assert (dists >= 0).all() and (dists <= 4 + 1e-6).all()


# ---------------------------------------------------------------- library second opinions
@pytest.mark.parametrize("dtype", ["f32", "u8"])
def test_against_scipy_cdist_and_lexsort(dtype):
    rng = np.random.default_rng(5)
    n, nlist, d, k = 37, 53, 19, 11  # all different: a transposed operand cannot pass
    if dtype == "u8":
        x = rng.integers(0, 256, (n, d)).astype(np.uint8)
        c = (rng.integers(0, 256, (nlist, d))).astype(np.float32)
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
        c = rng.standard_normal((nlist, d)).astype(np.float32)
    D = ssd.cdist(x.astype(np.float64), c.astype(np.float64), "sqeuclidean")
    ids, dists, nxt = oracle.route(x, c, k)
    for i in range(n):
        order = np.lexsort((np.arange(nlist), D[i]))  # by distance, then by id
        assert ids[i].tolist() == order[:k].tolist()
        np.testing.assert_allclose(dists[i], D[i, order[:k]], rtol=1e-12, atol=1e-9)
        assert nxt[i] == pytest.approx(D[i, order[k]], rel=1e-12)


def test_ties_resolved_by_lower_id_with_many_duplicates():
    # few distinct integer points -> many exact ties; lexsort on exact integers is the reference
    rng = np.random.default_rng(11)
    x = rng.integers(0, 3, (20, 4)).astype(np.uint8)
    c = rng.integers(0, 3, (64, 4)).astype(np.float32)
    D = ((x[:, None, :].astype(np.int64) - c[None].astype(np.int64)) ** 2).sum(-1)
    ids, dists, _ = oracle.route(x, c, 17)
    for i in range(20):
        order = np.lexsort((np.arange(64), D[i]))
        assert ids[i].tolist() == order[:17].tolist()
        assert dists[i].tolist() == D[i, order[:17]].astype(np.float64).tolist()
    assert any(len(set(D[i].tolist())) < 20 for i in range(20))  # ties really occur


# ---------------------------------------------------------------- brute force on Eq. 1
def test_eq1_subset_argmin_is_k_smallest():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((6, 5)).astype(np.float32)
    c = rng.standard_normal((8, 5)).astype(np.float32)
    D = ssd.cdist(x.astype(np.float64), c.astype(np.float64), "sqeuclidean")
    for k in (1, 3, 5):
        ids, _, _ = oracle.route(x, c, k)
        for i in range(6):
            best = min(itertools.combinations(range(8), k), key=lambda s: sum(D[i, j] for j in s))
            assert set(ids[i].tolist()) == set(best)


# ---------------------------------------------------------------- invariants
def test_k_equals_nlist_gives_sorted_permutation():
    q, c = synth.routing_inputs(synth.C0, nq=9, nlist=33)
    ids, dists, nxt = oracle.route(q, c, 33)
    assert np.isinf(nxt).all()
    for i in range(9):
        assert sorted(ids[i].tolist()) == list(range(33))
        assert (np.diff(dists[i]) >= 0).all()


def test_centroid_as_query_finds_itself_lowest_id_among_duplicates():
    _, c = synth.routing_inputs(synth.C0, nq=1, nlist=40)
    c[25] = c[7]  # duplicate: both at distance zero from query 7 and query 25
    ids, dists, _ = oracle.route(c, c, 2)
    assert (dists[:, 0] == 0).all()
    want = np.arange(40); want[25] = 7
    assert ids[:, 0].tolist() == want.tolist()
    assert ids[7].tolist() == [7, 25] and ids[25].tolist() == [7, 25]


def test_permuting_centroids_permutes_ids():
    q, c = synth.routing_inputs(synth.C0, nq=30, nlist=100)
    perm = np.random.default_rng(1).permutation(100)
    ids_a, d_a, _ = oracle.route(q, c, 10)
    ids_b, d_b, _ = oracle.route(q, c[perm], 10)
    assert (perm[ids_b] == ids_a).all()  # continuous data: no ties
    assert (d_a == d_b).all()


def test_prefix_property_and_assign_is_route_k1():
    q, c = synth.routing_inputs(synth.C1, nq=25, nlist=300)
    ids5, d5, _ = oracle.route(q, c, 5)
    ids6, d6, nxt5 = oracle.route(q, c, 6)[0], oracle.route(q, c, 6)[1], oracle.route(q, c, 5)[2]
    assert (ids6[:, :5] == ids5).all() and (d6[:, :5] == d5).all()
    assert (d6[:, 5] == nxt5).all()
    a_ids, a_d = oracle.assign(q, c)
    assert (a_ids == ids5[:, 0]).all() and (a_d == d5[:, 0]).all()


def test_translation_and_scaling_on_integers():
    q, c = synth.integer_case(12, 40, 6, seed=0, hi=100)
    ids, dists, _ = oracle.route(q, c, 7)
    shift = np.array([5, 0, 17, 3, 9, 1])
    ids_t, d_t, _ = oracle.route((q + shift).astype(np.uint8), c + shift.astype(np.float32), 7)
    assert (ids_t == ids).all() and (d_t == dists).all()
    ids_s, d_s, _ = oracle.route((2 * q).astype(np.uint8), 2 * c, 7)
    assert (ids_s == ids).all() and (d_s == 4 * dists).all()


def test_pair_dists_and_sqnorms():
    rng = np.random.default_rng(8)
    x = rng.integers(0, 256, (10, 12)).astype(np.uint8)
    c = rng.standard_normal((14, 12)).astype(np.float32) * 50
    rows = rng.integers(0, 10, 30); cols = rng.integers(0, 14, 30)
    got = oracle.pair_dists(x, c, rows, cols)
    want = ((x[rows].astype(np.float64) - c[cols].astype(np.float64)) ** 2).sum(1)
    np.testing.assert_allclose(got, want, rtol=1e-13)
    np.testing.assert_allclose(oracle.sqnorms(x), (x.astype(np.float64) ** 2).sum(1), rtol=1e-15)
    np.testing.assert_allclose(oracle.sqnorms(c), (c.astype(np.float64) ** 2).sum(1), rtol=1e-13)


# ---------------------------------------------------------------- Lloyd update
def test_update_against_bincount_and_totals():
    rng = np.random.default_rng(2)
    n, d, nlist = 500, 9, 23
    x = rng.integers(0, 256, (n, d)).astype(np.uint8)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    sums, counts, ok = oracle.update(x, ids, nlist)
    assert ok
    assert counts.sum() == n
    assert (counts == np.bincount(ids, minlength=nlist)).all()
    want = np.zeros((nlist, d)); np.add.at(want, ids, x.astype(np.float64))
    assert (sums == want).all()  # integers: exact
    assert (sums.sum(0) == x.astype(np.int64).sum(0)).all()


def test_update_accumulates_singletons_and_bad_ids():
    x = np.array([[1.5, 2.0], [3.0, -4.0], [10.0, 10.0]], np.float32)
    sums, counts, ok = oracle.update(x[:2], np.array([2, 0], np.int32), 3)
    assert ok and counts.tolist() == [1, 0, 1]
    assert sums.tolist() == [[3.0, -4.0], [0.0, 0.0], [1.5, 2.0]]  # one member -> the row itself
    sums, counts, ok = oracle.update(x[2:], np.array([2], np.int32), 3, sums, counts)  # second chunk
    assert ok and counts.tolist() == [1, 0, 2] and sums[2].tolist() == [11.5, 12.0]
    s2, c2, ok2 = oracle.update(x, np.array([0, 7, -1], np.int32), 3)
    assert not ok2 and c2.tolist() == [1, 0, 0] and s2[0].tolist() == [1.5, 2.0]


def test_finalize_mean_and_empty_list_keeps_old():
    sums = np.array([[3.0, 6.0], [0.0, 0.0], [1.0, 2.0]])
    counts = np.array([3, 0, 4], np.int64)
    old = np.array([[9, 9], [7, 8], [9, 9]], np.float32)
    new = oracle.finalize(sums, counts, old)
    assert new.tolist() == [[1.0, 2.0], [7.0, 8.0], [0.25, 0.5]]
    assert old.tolist() == [[9, 9], [7, 8], [9, 9]]


def test_lloyd_inertia_monotone_and_matches_stepwise_pieces():
    x = synth.sift_like_rows(0, rows=3000)
    init = x[synth.init_sample(3000, 50)].astype(np.float32)
    c, ids, inertia = oracle.lloyd(x, init, 5)
    assert (np.diff(inertia) <= 1e-9 * inertia[0]).all()
    # replay with the separate pieces
    cc = init.copy()
    for it in range(5):
        a_ids, a_d = oracle.assign(x, cc)
        assert a_d.sum() == pytest.approx(inertia[it], rel=1e-12)
        s, n_, ok = oracle.update(x, a_ids, 50)
        cc = oracle.finalize(s, n_, cc)
    assert (cc == c).all() and (a_ids == ids).all()


def test_lloyd_every_row_its_own_list():
    rng = np.random.default_rng(4)
    x = rng.permutation(200)[:40, None].astype(np.float32) * np.ones((1, 3), np.float32)  # distinct rows
    c, ids, inertia = oracle.lloyd(x, x.copy(), 2)
    assert (inertia == 0).all() and ids.tolist() == list(range(40)) and (c == x).all()


# ---------------------------------------------------------------- cluster-major reorder
def test_reorder_hand_case_and_stable_argsort():
    ids = np.array([2, 0, 2, 1, 0, 2], np.int32)
    offsets, order = oracle.reorder(ids, 4)
    assert offsets.tolist() == [0, 2, 3, 6, 6]        # list 3 is empty
    assert order.tolist() == [1, 4, 3, 0, 2, 5]       # input order kept inside each list
    rng = np.random.default_rng(6)
    ids = rng.integers(0, 37, 5000).astype(np.int32)
    offsets, order = oracle.reorder(ids, 37)
    assert (order == np.argsort(ids, kind="stable")).all()
    assert (np.diff(offsets) == np.bincount(ids, minlength=37)).all() and offsets[-1] == 5000
    with pytest.raises(ValueError):
        oracle.reorder(np.array([0, 5], np.int32), 5)


# ---------------------------------------------------------------- assignment within given candidates
def test_candidate_assignment_hand_case_and_ties():
    # points on a line; candidates given explicitly.  x = 5: candidates {0 at 0, 2 at 9, 3 at 1} ->
    # distances 25, 16, 16: tie between ids 2 and 3 -> id 2.  x = 0 with candidates {3, 3}: id 3, 1.
    c = np.array([[0.0], [100.0], [9.0], [1.0]], np.float32)
    x = np.array([[5.0], [0.0]], np.float32)
    cand = np.array([[0, 2, 3], [3, 3, 3]], np.int32)
    ids, d = oracle.assign_candidates(x, c, cand)
    assert ids.tolist() == [2, 3] and d.tolist() == [16.0, 1.0]
    # order of the candidates does not matter, nor do repeats
    ids2, d2 = oracle.assign_candidates(x, c, np.array([[3, 0, 2], [3, 3, 3]], np.int32))
    assert ids2.tolist() == [2, 3] and d2.tolist() == [16.0, 1.0]


def test_candidate_assignment_against_numpy_and_full_assignment():
    rng = np.random.default_rng(21)
    n, nlist, d, m = 400, 300, 24, 8
    x = rng.integers(0, 256, (n, d)).astype(np.uint8)
    c = rng.normal(120, 40, (nlist, d)).astype(np.float32)
    cand = rng.integers(0, nlist, (n, m)).astype(np.int32)
    ids, dist = oracle.assign_candidates(x, c, cand)
    gathered = c[cand].astype(np.float64)                         # [n, m, d]
    ref = ((x.astype(np.float64)[:, None, :] - gathered) ** 2).sum(-1)
    pick = np.array([min(range(m), key=lambda p: (ref[i, p], cand[i, p])) for i in range(n)])
    assert (ids == cand[np.arange(n), pick]).all()
    assert np.allclose(dist, ref[np.arange(n), pick], rtol=1e-12)
    # if the true nearest centroid is among the candidates the result is the full assignment
    full_ids, full_d = oracle.assign(x, c)
    cand[:, 3] = full_ids
    ids, dist = oracle.assign_candidates(x, c, cand)
    assert (ids == full_ids).all() and (dist == full_d).all()
    # all centroids as candidates: the same again
    every = np.tile(np.arange(nlist, dtype=np.int32), (n, 1))
    ids, dist = oracle.assign_candidates(x, c, every)
    assert (ids == full_ids).all() and (dist == full_d).all()
    bad = cand.copy(); bad[0, 0] = nlist
    with pytest.raises(ValueError):
        oracle.assign_candidates(x, c, bad)
