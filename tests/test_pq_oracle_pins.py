"""Pins of the residual-PQ oracle against what the paper's definitions and the mathematics fix
(Eq. 3 encoding, Eq. 4 lookup table, Eq. 5 ADC estimate, Sec. 4.3 / 4.4 candidate reduction):
hand-computed values, closed forms, the decode identity in fp64, integer-exact data, fp64 arg-min
and lexsort cross-checks, and invariants.  None of the expected values comes from the oracle."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_08751_b200 import synth


def _far_codebooks(pq_m, dsub):
    # every codeword far away (1000, 1000, ...) so that the few set by a test decide everything
    return np.full((pq_m, 256, dsub), 1000.0, np.float32)


def test_hand_computed_table_codes_and_estimates():
    # d = 4, two subspaces of two coordinates.  Point x = (7, 1, 2, 9), centroid (4, 5, 2, 4):
    # residual (3, -4 | 0, 5).  Subspace 0 codewords: #3 = (0, 0) -> 9 + 16 = 25, #7 = (3, -1) -> 9,
    # #200 = (2, -4) -> 1.  Subspace 1: #0 = (0, 0) -> 25, #9 = (1, 5) -> 1, #10 = (-1, 5) -> 1 (tie).
    cb = _far_codebooks(2, 2)
    cb[0, 3] = (0, 0); cb[0, 7] = (3, -1); cb[0, 200] = (2, -4)
    cb[1, 0] = (0, 0); cb[1, 9] = (1, 5); cb[1, 10] = (-1, 5)
    c = np.array([[0, 0, 0, 0], [4, 5, 2, 4]], np.float32)
    x = np.array([[7, 1, 2, 9]], np.uint8)
    lut = O.pq_lut(np.array([3, -4, 0, 5], np.float32), cb)
    assert lut[0, 3] == 25 and lut[0, 7] == 9 and lut[0, 200] == 1
    assert lut[1, 0] == 25 and lut[1, 9] == 1 and lut[1, 10] == 1
    assert lut[0, 1] == (1000 - 3) ** 2 + (1000 + 4) ** 2
    codes = O.pq_encode(x, np.array([1], np.int32), c, cb)
    assert codes.tolist() == [[200, 9]]  # the tie in subspace 1 goes to the lower index
    # a query equal to the point, probing list 1 which stores codes (200, 9), (7, 0), (3, 10):
    stored = np.array([[200, 9], [7, 0], [3, 10]], np.uint8)
    offsets = np.array([0, 0, 3], np.int64)
    pos, est, cnt = O.pq_search(x, c, np.array([[1]], np.int32), offsets, stored, cb, 2)
    assert cnt.tolist() == [3]
    assert pos.tolist() == [[0, 2]] and est.tolist() == [[2.0, 26.0]]  # 1+1, 25+1; (9+25 = 34 dropped)
    assert O.pq_adc(lut, stored).tolist() == [2.0, 34.0, 26.0]


def test_exact_codeword_closed_form_and_duplicates():
    # if a residual sub-vector IS codeword j, the code is j and the table entry is 0; a duplicate
    # of that codeword at a higher index never wins
    rng = np.random.default_rng(1)
    pq_m, dsub, d = 4, 3, 12
    cb = rng.normal(0, 5, (pq_m, 256, dsub)).astype(np.float32)
    cb[:, 250] = cb[:, 17]  # duplicates
    c = rng.normal(0, 1, (5, d)).astype(np.float32)
    want = rng.integers(0, 250, size=(40, pq_m))
    want[:10, 0] = 17
    ids = rng.integers(0, 5, 40).astype(np.int32)
    # build x so that x - c is exactly representable: use integer centroids and codebooks
    c = np.rint(c * 4)
    cb = np.rint(cb)
    cb[:, 250] = cb[:, 17]
    # make codewords distinct apart from the planted duplicate
    for m in range(pq_m):
        cb[m, :, 0] += np.arange(256) * 64
        cb[m, 250] = cb[m, 17]
    x = (c[ids] + np.concatenate([cb[m, want[:, m]] for m in range(pq_m)], axis=1)).astype(np.float32)
    codes = O.pq_encode(x, ids, c.astype(np.float32), cb.astype(np.float32))
    assert (codes == want).all()
    lut = O.pq_lut((x[0] - c[ids[0]]).astype(np.float32), cb.astype(np.float32))
    assert all(lut[m, want[0, m]] == 0 for m in range(pq_m))


def test_encode_matches_fp64_argmin_away_from_near_ties():
    rng = np.random.default_rng(2)
    n, nlist, d, pq_m = 300, 20, 32, 8
    dsub = d // pq_m
    c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
    cb = synth.pq_codebooks(pq_m, dsub, 0.3, seed=2)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    x = (c[ids] + rng.normal(0, 0.3, (n, d))).astype(np.float32)
    codes = O.pq_encode(x, ids, c, cb)
    r = x.astype(np.float64) - c[ids].astype(np.float64)
    for m in range(pq_m):
        dist = ((r[:, None, m * dsub:(m + 1) * dsub] - cb[m][None].astype(np.float64)) ** 2).sum(-1)
        ref = dist.argmin(1)
        bad = codes[:, m] != ref
        # any disagreement must be a near-tie at fp32 resolution
        gap = np.abs(dist[np.arange(n), codes[:, m]] - dist[np.arange(n), ref])
        assert (gap[bad] <= 1e-5 * dist[np.arange(n), ref][bad]).all()
        assert bad.mean() < 0.02


def test_adc_estimate_is_the_distance_to_the_decoded_vector():
    # sum_m |r_q^(m) - p_m[a_m]|^2 = |q - (c + decode(a))|^2: a second opinion in fp64 numpy
    rng = np.random.default_rng(3)
    nlist, d, pq_m, n = 6, 24, 6, 200
    dsub = d // pq_m
    c = rng.normal(0, 2, (nlist, d)).astype(np.float32)
    cb = synth.pq_codebooks(pq_m, dsub, 1.0, seed=3)
    codes = rng.integers(0, 256, (n, pq_m)).astype(np.uint8)
    q = rng.normal(0, 2, (d,)).astype(np.float32)
    for l in range(nlist):
        lut = O.pq_lut(q - c[l], cb)
        est = O.pq_adc(lut, codes)
        decoded = np.concatenate([cb[m, codes[:, m]] for m in range(pq_m)], axis=1).astype(np.float64)
        ref = ((q.astype(np.float64) - (c[l].astype(np.float64) + decoded)) ** 2).sum(1)
        assert np.allclose(est, ref, rtol=2e-6, atol=1e-6)


def _integer_problem(seed, nq=12, nlist=30, n=4000, d=16, pq_m=4, nprobe=5):
    rng = np.random.default_rng(seed)
    dsub = d // pq_m
    c = rng.integers(0, 200, (nlist, d)).astype(np.float32)
    cb = synth.pq_codebooks(pq_m, dsub, 20.0, seed=seed, integer=True)
    ids, offsets = synth.skewed_list_ids(n, nlist, seed)
    x = synth.rows_near(c, ids, 20.0, seed, "u8")
    q = rng.integers(0, 256, (nq, d)).astype(np.uint8)
    probes = synth.distinct_probes(nq, nlist, nprobe, seed)
    return q, c, cb, ids, offsets, x, probes


def test_integer_data_equals_int64_arithmetic_bit_for_bit():
    # uint8 points, integer centroids and codewords: every difference, square and sum is an
    # integer < 2^24, so float32 in any order must equal int64 arithmetic exactly, ties included
    q, c, cb, ids, offsets, x, probes = _integer_problem(4)
    pq_m, dsub = cb.shape[0], cb.shape[2]
    ci, cbi = c.astype(np.int64), cb.astype(np.int64)
    r = x.astype(np.int64) - ci[ids]
    ref_codes = np.empty((len(x), pq_m), np.uint8)
    for m in range(pq_m):
        dist = ((r[:, None, m * dsub:(m + 1) * dsub] - cbi[m][None]) ** 2).sum(-1)
        ref_codes[:, m] = dist.argmin(1)  # numpy argmin returns the first minimum = lower index
    codes = O.pq_encode(x, ids, c, cb)
    assert (codes == ref_codes).all()
    n_rerank = 50
    pos, est, cnt = O.pq_search(q, c, probes, offsets, codes, cb, n_rerank)
    for b in range(len(q)):
        cand_pos, cand_est = [], []
        for l in probes[b]:
            rq = q[b].astype(np.int64) - ci[l]
            lut = np.stack([((rq[m * dsub:(m + 1) * dsub][None] - cbi[m]) ** 2).sum(-1) for m in range(pq_m)])
            seg = codes[offsets[l]:offsets[l + 1]]
            cand_est.append(lut[np.arange(pq_m)[None], seg].sum(1))
            cand_pos.append(np.arange(offsets[l], offsets[l + 1]))
        cand_pos, cand_est = np.concatenate(cand_pos), np.concatenate(cand_est)
        assert cand_est.max() < 2 ** 24
        order = np.lexsort((cand_pos, cand_est))[:n_rerank]
        assert cnt[b] == len(cand_pos)
        k = len(order)
        assert (pos[b, :k] == cand_pos[order]).all()
        assert (est[b, :k] == cand_est[order].astype(np.float32)).all()
        assert (pos[b, k:] == -1).all() and np.isinf(est[b, k:]).all()


def test_search_matches_fp64_lexsort_inside_rounding():
    rng = np.random.default_rng(5)
    nq, nlist, n, d, pq_m, nprobe, n_rerank = 8, 40, 6000, 32, 8, 6, 64
    dsub = d // pq_m
    c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
    cb = synth.pq_codebooks(pq_m, dsub, 0.3, seed=5)
    ids, offsets = synth.skewed_list_ids(n, nlist, 5)
    x = synth.rows_near(c, ids, 0.3, 5)
    codes = O.pq_encode(x, ids, c, cb)
    q = rng.normal(0, 1, (nq, d)).astype(np.float32)
    probes = synth.distinct_probes(nq, nlist, nprobe, 5)
    pos, est, cnt = O.pq_search(q, c, probes, offsets, codes, cb, n_rerank)
    decoded = np.concatenate([cb[m, codes[:, m]] for m in range(pq_m)], axis=1).astype(np.float64)
    for b in range(nq):
        cand = np.concatenate([np.arange(offsets[l], offsets[l + 1]) for l in probes[b]])
        ref = ((q[b].astype(np.float64) - (c[ids[cand]].astype(np.float64) + decoded[cand])) ** 2).sum(1)
        order = np.lexsort((cand, ref))
        kth = ref[order[n_rerank - 1]]
        tol = 4e-6 * kth
        got = set(pos[b].tolist())
        assert len(got) == n_rerank and got <= set(cand.tolist())
        assert set(cand[ref < kth - tol].tolist()) <= got          # clear winners are all there
        e64 = dict(zip(cand.tolist(), ref.tolist()))
        assert all(e64[p] <= kth + tol for p in got)                 # nothing clearly worse got in
        assert np.allclose(est[b], [e64[p] for p in pos[b]], rtol=4e-6, atol=1e-7)
        assert (np.diff(est[b]) >= 0).all()


def test_prefix_padding_and_translation_invariants():
    q, c, cb, ids, offsets, x, probes = _integer_problem(6, nq=6, nlist=12, n=300, nprobe=3)
    codes = O.pq_encode(x, ids, c, cb)
    big = O.pq_search(q, c, probes, offsets, codes, cb, 400)   # more slots than candidates
    small = O.pq_search(q, c, probes, offsets, codes, cb, 30)
    for b in range(len(q)):
        cnt = int(big[2][b])
        assert cnt == sum(offsets[l + 1] - offsets[l] for l in probes[b]) and cnt < 400
        assert (big[0][b, cnt:] == -1).all() and (big[0][b, :cnt] >= 0).all()
        assert sorted(big[0][b, :cnt].tolist()) == sorted(
            p for l in probes[b] for p in range(offsets[l], offsets[l + 1]))
        k = min(30, cnt)
        assert (small[0][b, :k] == big[0][b, :k]).all() and (small[1][b, :k] == big[1][b, :k]).all()
    # shifting queries, points and centroids by the same integer vector changes no residual
    shift = np.arange(c.shape[1]) % 7
    q2 = (q.astype(np.int64) + shift).astype(np.float32)
    x2 = (x.astype(np.int64) + shift).astype(np.float32)
    c2 = c + shift.astype(np.float32)
    assert (O.pq_encode(x2, ids, c2, cb) == codes).all()
    moved = O.pq_search(q2, c2, probes, offsets, codes, cb, 30)
    assert (moved[0] == small[0]).all() and (moved[1] == small[1]).all()
    # the order of a query's probes does not matter
    flipped = O.pq_search(q, c, probes[:, ::-1].copy(), offsets, codes, cb, 30)
    assert (flipped[0] == small[0]).all() and (flipped[1] == small[1]).all()


def test_bad_arguments_are_refused():
    q, c, cb, ids, offsets, x, probes = _integer_problem(7, nq=2, nlist=5, n=50, nprobe=2)
    bad = ids.copy(); bad[3] = 99
    with pytest.raises(ValueError):
        O.pq_encode(x, bad, c, cb)
    codes = O.pq_encode(x, ids, c, cb)
    badp = probes.copy(); badp[0, 0] = -1
    with pytest.raises(ValueError):
        O.pq_search(q, c, badp, offsets, codes, cb, 4)


def test_residuals_against_numpy():
    rng = np.random.default_rng(31)
    c = rng.normal(0, 3, (9, 12)).astype(np.float32)
    ids = rng.integers(0, 9, 50).astype(np.int32)
    for x in (rng.integers(0, 256, (50, 12)).astype(np.uint8), rng.integers(-128, 128, (50, 12)).astype(np.int8),
              rng.normal(0, 3, (50, 12)).astype(np.float32)):
        r = O.residuals(x, ids, c)
        assert r.dtype == np.float32 and (r == (x.astype(np.float32) - c[ids])).all()
    # a point equal to its centroid has a zero residual; the encoder then picks the codeword nearest 0
    x = c[ids].copy()
    assert (O.residuals(x, ids, c) == 0).all()
    with pytest.raises(ValueError):
        O.residuals(x, np.full(50, 9, np.int32), c)
