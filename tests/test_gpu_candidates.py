"""GPU parity of the candidate-restricted assignment (exact distance within 2-8 given candidate
centroids per vector) against the CPU oracle, through the C-ABI binding."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import synth

pytestmark = pytest.mark.gpu


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run(x, c, cand):
    ids, d = B.ivf_assign_candidates(_t(x), _t(c), _t(cand))
    B.ivf_check()
    return ids.cpu().numpy(), d.cpu().numpy()


@pytest.mark.parametrize("n,nlist,d,m", [(1, 1, 4, 1), (1000, 500, 128, 8), (777, 3000, 128, 2), (300, 64, 256, 13),
                                         (513, 900, 96, 5), (200, 50, 100, 8), (65, 10, 16, 3)])
def test_integer_inputs_are_bit_identical(n, nlist, d, m):
    # uint8 points and integer centroids: every difference, square and sum is exact in fp32, so ids
    # (ties included: few distinct values) and distances must equal the fp64 oracle exactly
    rng = np.random.default_rng(n + d + m)
    x = rng.integers(0, 8, (n, d)).astype(np.uint8)
    c = rng.integers(0, 8, (nlist, d)).astype(np.float32)
    cand = rng.integers(0, nlist, (n, m)).astype(np.int32)
    ids, dist = _run(x, c, cand)
    want_ids, want_d = O.assign_candidates(x, c, cand)
    assert (ids == want_ids).all()
    assert (dist.astype(np.float64) == want_d).all()


@pytest.mark.parametrize("n,nlist,d,m,dtype", [(2000, 4000, 128, 8, "u8"), (1500, 3000, 96, 8, "f32"), (900, 2000, 100, 2, "f32")])
def test_real_valued_inputs_within_fp32_rounding(n, nlist, d, m, dtype):
    # fp32 direct-difference sums of d terms: relative error below d * 2^-23, checked at 1e-5; the
    # chosen id may differ from the oracle's only where the two distances are that close
    if dtype == "u8":
        c = synth.sift_like_centroids(nlist, d)
        x = synth.sift_like_rows(3, rows=n, d=d)
    else:
        rng = np.random.default_rng(5)
        c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
        x = rng.normal(0, 1, (n, d)).astype(np.float32)
    near, _, _ = O.route(x, c, m)
    cand = near[:, ::-1].copy()  # the true nearest comes last
    ids, dist = _run(x, c, cand)
    want_ids, want_d = O.assign_candidates(x, c, cand)
    got_true = O.pair_dists(x, c, np.arange(n), ids)
    tol = 1e-5 * np.maximum(want_d, 1e-30)
    assert (np.abs(dist - got_true) <= 1e-5 * np.maximum(got_true, 1e-30)).all()
    assert (got_true <= want_d + tol).all()
    assert (ids == want_ids).mean() > 0.999
    # with the true nearest among the candidates this is the full assignment
    full_ids, _ = O.assign(x, c)
    assert (want_ids == full_ids).all()


def test_chunk_sized_batch_every_row_checked():
    # the assignment batch of the ultra-fast mode (1,048,576 rows, Table 3) against 65,536 centroids
    n, nlist, d, m = 1 << 20, 65536, 128, 8
    x = synth.sift_like_rows(0, rows=n, d=d)
    c = synth.sift_like_centroids(nlist, d)
    cand = np.random.default_rng(9).integers(0, nlist, (n, m)).astype(np.int32)
    ids, dist = _run(x, c, cand)
    want_ids, want_d = O.assign_candidates(x, c, cand)
    got_true = O.pair_dists(x, c, np.arange(n), ids)
    assert (np.abs(dist - got_true) <= 1e-5 * got_true).all()
    assert (got_true <= want_d * (1 + 1e-5)).all()
    assert (ids == want_ids).mean() > 0.9999


def test_bad_candidate_is_skipped_and_flagged():
    rng = np.random.default_rng(2)
    x = rng.integers(0, 256, (40, 32)).astype(np.uint8)
    c = rng.integers(0, 256, (20, 32)).astype(np.float32)
    cand = rng.integers(0, 20, (40, 4)).astype(np.int32)
    good_ids, _ = O.assign_candidates(x, c, cand[:, 1:])
    cand[:, 0] = 20
    cand[7, :] = -1
    ids, dist = B.ivf_assign_candidates(_t(x), _t(c), _t(cand))
    with pytest.raises(B.IvfError) as e:
        B.ivf_check()
    assert e.value.code == B.IVF_ERR_BAD_ID
    ids, dist = ids.cpu().numpy(), dist.cpu().numpy()
    keep = np.arange(40) != 7
    assert (ids[keep] == good_ids[keep]).all()
    assert ids[7] == -1 and np.isinf(dist[7])
