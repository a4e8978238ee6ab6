"""GPU parity of the residual-PQ chain (encode, set-up, chunked ADC scan, group and query merge)
against the CPU oracle, through the C-ABI binding.  The oracle computes in the paper's fp32 with a
stated operation order, so codes, kept positions and estimates must match bit for bit.  Every
oracle input comes from the seeded generators or from the oracle itself, never from the GPU."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _problem(seed, n, nlist, d, pq_m, dtype, nq, nprobe, sigma=1.0, integer=False):
    rng = np.random.default_rng(1000 + seed)
    dsub = d // pq_m
    if dtype == "u8":
        c = rng.uniform(20, 230, (nlist, d)).astype(np.float32)
        if integer:
            c = np.rint(c)
        scale = 20.0
        q = rng.integers(0, 256, (nq, d)).astype(np.uint8)
    else:
        c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
        scale = 0.3
        q = (c[rng.integers(0, nlist, nq)] + rng.normal(0, 0.4, (nq, d))).astype(np.float32)
    cb = synth.pq_codebooks(pq_m, dsub, scale, seed, integer=integer)
    ids, offsets = synth.skewed_list_ids(n, nlist, seed, sigma)
    x = synth.rows_near(c, ids, scale, seed, dtype)
    probes = synth.distinct_probes(nq, nlist, nprobe, seed)
    return q, c, cb, ids, offsets, x, probes


SHAPES = [
    # n, nlist, d, pq_m, dtype
    (3000, 40, 128, 32, "u8"),    # SIFT-shaped, 100M-scale code size (Table 2)
    (3000, 40, 128, 16, "u8"),    # SIFT-shaped, 1B-scale code size
    (2500, 30, 96, 32, "f32"),    # DEEP-shaped, sub-vectors of 3
    (2500, 30, 96, 16, "f32"),    # DEEP-shaped, sub-vectors of 6
    (2000, 25, 100, 20, "f32"),   # SPACEV-shaped width, 4-byte code path
    (2000, 25, 100, 50, "f32"),   # SPACEV-shaped width, byte code path
    (500, 7, 8, 8, "f32"),        # one coordinate per subspace
    (500, 7, 16, 1, "u8"),        # a single subspace
]


@pytest.mark.parametrize("n,nlist,d,pq_m,dtype", SHAPES)
def test_encode_is_bit_identical(n, nlist, d, pq_m, dtype):
    q, c, cb, ids, offsets, x, probes = _problem(1, n, nlist, d, pq_m, dtype, 4, 2)
    want = O.pq_encode(x, ids, c, cb)
    got = B.ivf_pq_encode(_t(x), _t(ids), _t(c), _t(cb))
    B.ivf_check()
    assert (got.cpu().numpy() == want).all()


def _check_search(q, c, cb, offsets, codes, probes, n_rerank, vec_ids=None):
    want_pos, want_est, want_cnt = O.pq_search(q, c, probes, offsets, codes, cb, n_rerank)
    got_pos, got_est, got_cnt = B.ivf_pq_search(_t(q), _t(c), _t(probes), _t(offsets), _t(codes), _t(cb), n_rerank,
                                                vec_ids=None if vec_ids is None else _t(vec_ids))
    B.ivf_check()
    got_pos, got_est, got_cnt = got_pos.cpu().numpy(), got_est.cpu().numpy(), got_cnt.cpu().numpy()
    assert (got_cnt == want_cnt).all()
    if vec_ids is not None:
        want_pos = np.where(want_pos >= 0, vec_ids[np.maximum(want_pos, 0)], -1)
    assert (got_pos == want_pos).all()
    assert (got_est.view(np.uint32) == want_est.view(np.uint32)).all()


@pytest.mark.parametrize("n,nlist,d,pq_m,dtype", SHAPES)
@pytest.mark.parametrize("nq,nprobe,n_rerank", [(1, 1, 16), (9, 5, 64), (37, 7, 512)])
def test_search_is_bit_identical(n, nlist, d, pq_m, dtype, nq, nprobe, n_rerank):
    nprobe = min(nprobe, nlist)
    q, c, cb, ids, offsets, x, probes = _problem(2, n, nlist, d, pq_m, dtype, nq, nprobe)
    codes = O.pq_encode(x, ids, c, cb)
    _check_search(q, c, cb, offsets, codes, probes, n_rerank)


@pytest.mark.parametrize("n_rerank", [1, 100, 512, 1024])
def test_long_lists_many_buffer_cuts_and_ties(n_rerank):
    # a few very long lists (many chunks per group, the buffer is cut back again and again) and
    # integer data, where equal estimates are plentiful: the (estimate, position) order must hold
    q, c, cb, ids, offsets, x, probes = _problem(3, 60000, 12, 32, 8, "u8", 5, 6, sigma=1.5, integer=True)
    codes = O.pq_encode(x, ids, c, cb)
    assert (offsets[1:] - offsets[:-1]).max() > 8 * 1024
    _check_search(q, c, cb, offsets, codes, probes, n_rerank)


@pytest.mark.parametrize("groups", [1, 2, 7, 256, -2, -8])  # negative: the scan kernel that reads the codebook through L1
def test_every_group_count_gives_the_same_result(groups):
    # the chunks of a query are dealt to `groups` CTAs whose survivors the query merge combines:
    # in shared memory when they fit, by a select over the group outputs when they do not
    q, c, cb, ids, offsets, x, probes = _problem(4, 150000, 60, 64, 16, "f32", 6, 16, sigma=1.2)
    codes = O.pq_encode(x, ids, c, cb)
    B.ivf_debug_set_pq_groups(groups)
    try:
        _check_search(q, c, cb, offsets, codes, probes, 200)
        _check_search(q[:2], c, cb, offsets, codes, probes[:2], 1024)
    finally:
        B.ivf_debug_set_pq_groups(0)


@pytest.mark.parametrize("d,pq_m", [(128, 32), (64, 32)])  # sub-vectors of 4 and of 2
@pytest.mark.parametrize("groups", [0, -2])
def test_codebook_on_any_four_byte_boundary(d, pq_m, groups):
    # the table build reads these widths with vector loads when the codebook starts on a 16-byte
    # boundary and from a coordinate-major copy otherwise: same candidates and estimates either way
    q, c, cb, ids, offsets, x, probes = _problem(21, 30000, 50, d, pq_m, "u8", 11, 9)
    codes = O.pq_encode(x, ids, c, cb)
    flat = torch.zeros(cb.size + 4, dtype=torch.float32, device=DEV)
    B.ivf_debug_set_pq_groups(groups)
    try:
        outs = []
        for shift in (0, 1, 2):
            view = flat[shift:shift + cb.size].view(cb.shape)
            view.copy_(_t(cb))
            assert (view.data_ptr() % 16 == 0) == (shift == 0)
            got = B.ivf_pq_search(_t(q), _t(c), _t(probes), _t(offsets), _t(codes), view, 128)
            outs.append([t.cpu().numpy() for t in got])
        for o in outs[1:]:
            for a, b in zip(outs[0], o):
                assert (a == b).all()
        _check_search(q, c, cb, offsets, codes, probes, 128)
    finally:
        B.ivf_debug_set_pq_groups(0)


def test_large_batch_one_group_per_query():
    q, c, cb, ids, offsets, x, probes = _problem(8, 40000, 300, 64, 16, "f32", 3000, 16)
    codes = O.pq_encode(x, ids, c, cb)
    _check_search(q, c, cb, offsets, codes, probes, 64)


def test_fewer_candidates_than_slots_empty_lists_and_identifier_map():
    q, c, cb, ids, offsets, x, probes = _problem(5, 400, 60, 32, 8, "f32", 20, 3, sigma=2.0)
    lens = offsets[1:] - offsets[:-1]
    assert (lens == 0).any()
    probes[0, :] = np.flatnonzero(lens == 0)[:1].tolist() + np.flatnonzero(lens > 0)[:2].tolist()
    probes[1, :] = np.argsort(lens)[:3]  # the three shortest lists
    codes = O.pq_encode(x, ids, c, cb)
    vec_ids = np.random.default_rng(0).permutation(len(x)).astype(np.int64) + 10 ** 10
    _check_search(q, c, cb, offsets, codes, probes, 512)
    _check_search(q, c, cb, offsets, codes, probes, 512, vec_ids=vec_ids)


def test_bad_ids_are_flagged_not_followed():
    q, c, cb, ids, offsets, x, probes = _problem(6, 300, 10, 32, 8, "f32", 4, 2)
    bad = ids.copy()
    bad[5] = 10
    codes = B.ivf_pq_encode(_t(x), _t(bad), _t(c), _t(cb))
    with pytest.raises(B.IvfError) as e:
        B.ivf_check()
    assert e.value.code == B.IVF_ERR_BAD_ID
    assert (codes[5].cpu().numpy() == 0).all()
    good = O.pq_encode(x, ids, c, cb)
    badp = probes.copy()
    badp[0, 0] = -3
    pos, est, cnt = B.ivf_pq_search(_t(q), _t(c), _t(badp), _t(offsets), _t(good), _t(cb), 8)
    with pytest.raises(B.IvfError):
        B.ivf_check()
    # the query simply loses that probe
    l = badp[0, 1]
    assert cnt[0].item() == offsets[l + 1] - offsets[l]


def test_argument_checks():
    q, c, cb, ids, offsets, x, probes = _problem(7, 100, 5, 32, 8, "f32", 2, 2)
    codes = _t(O.pq_encode(x, ids, c, cb))
    with pytest.raises(B.IvfError) as e:
        B.ivf_pq_search(_t(q), _t(c), _t(probes), _t(offsets), codes, _t(cb), 2000)
    assert e.value.code == B.IVF_ERR_UNSUPPORTED
    big = torch.zeros((64, 256, 4), dtype=torch.float32, device=DEV)  # d = 256: codebook does not fit
    with pytest.raises(B.IvfError) as e:
        B.ivf_pq_encode(torch.zeros((4, 256), device=DEV), torch.zeros(4, dtype=torch.int32, device=DEV),
                        torch.zeros((2, 256), device=DEV), big)
    assert e.value.code == B.IVF_ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype,d,pq_m", [("u8", 128, 32), ("f32", 96, 16)])
def test_full_size_batch_in_the_measured_configuration(dtype, d, pq_m):
    # the launch configuration the timing harness uses (2,048 queries, 64 probes chosen by the
    # oracle's own routing, N_rerank = 512, lists of about a thousand codes with a skewed length
    # distribution); every query is compared with the oracle bit for bit
    n, nlist, nq, nprobe, n_rerank = 1 << 20, 1024, 2048, 64, 512
    if dtype == "u8":
        c = synth.sift_like_centroids(nlist, d)
        q = synth.sift_like_queries(nq, d)
        scale = 20.0
    else:
        c = synth.deep_like_centroids(nlist, d)
        q = synth.deep_like_queries(nq, d)
        scale = 0.05
    cb = synth.pq_codebooks(pq_m, d // pq_m, scale, seed=11)
    ids, offsets = synth.skewed_list_ids(n, nlist, seed=11, sigma=0.7)
    x = synth.rows_near(c, ids, scale, 11, dtype)
    probes, _, _ = O.route(q, c, nprobe)
    want_codes = O.pq_encode(x, ids, c, cb)
    got_codes = B.ivf_pq_encode(_t(x), _t(ids), _t(c), _t(cb))
    B.ivf_check()
    assert (got_codes.cpu().numpy() == want_codes).all()
    _check_search(q, c, cb, offsets, want_codes, probes, n_rerank)


@pytest.mark.parametrize("nprobe", [257, 512])
def test_many_probes_take_the_single_team_kernel(nprobe):
    # more than 256 probes per query do not fit the two-team kernel's descriptor tables; 512 is the
    # largest probe count of the paper's sweep and of this library
    q, c, cb, ids, offsets, x, probes = _problem(9, 30000, 600, 64, 16, "f32", 5, nprobe, sigma=1.0)
    codes = O.pq_encode(x, ids, c, cb)
    _check_search(q, c, cb, offsets, codes, probes, 300)
    with pytest.raises(B.IvfError) as e:
        B.ivf_pq_search(_t(q), _t(c), _t(np.tile(probes, (1, 2))[:, :513].copy()), _t(offsets), _t(codes), _t(cb), 8)
    assert e.value.code in (B.IVF_ERR_UNSUPPORTED, B.IVF_ERR_INVALID_ARG)


def test_residuals_and_codebook_training_step_by_step():
    # residuals bit-identical; then every Lloyd step of the per-subspace training is compared with
    # the oracle fed the GPU's current codebook (so a tolerated near-tie cannot compound)
    from paper_2608_08751_b200 import pq_train
    import parity
    rng = np.random.default_rng(41)
    n, nlist, d, pq_m = 6000, 30, 32, 8
    dsub = d // pq_m
    c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
    ids, _ = synth.skewed_list_ids(n, nlist, seed=41)
    x = synth.rows_near(c, ids, 0.3, 41)
    res = B.ivf_pq_residuals(_t(x), _t(ids), _t(c))
    B.ivf_check()
    want = O.residuals(x, ids, c)
    assert (res.cpu().numpy().view(np.uint32) == want.view(np.uint32)).all()
    codebooks, inertia = pq_train.train_codebooks(_t(x), _t(ids), _t(c), pq_m, iters=4, seed=1, method="assign")
    B.ivf_check()
    assert codebooks.shape == (pq_m, 256, dsub)
    assert (np.diff(inertia.numpy(), axis=1) <= 1e-6 * inertia.numpy()[:, :-1]).all()  # Lloyd never gets worse
    # one more step on subspace 3, checked against the oracle: assignment inside the tolerance band,
    # sums and counts for the GPU's ids, means
    sub = np.ascontiguousarray(want[:, 3 * dsub:4 * dsub])
    cb = codebooks[3].clone()
    sums = torch.zeros((256, dsub), dtype=torch.float32, device="cuda")
    counts = torch.zeros((256,), dtype=torch.int64, device="cuda")
    a_ids = torch.empty((n,), dtype=torch.int32, device="cuda")
    a_d = torch.empty((n,), dtype=torch.float32, device="cuda")
    B.ivf_assign_update(_t(sub), cb, sums, counts, a_ids, a_d)
    B.ivf_check()
    g = a_ids.cpu().numpy()
    parity.check_route(sub, codebooks[3].cpu().numpy(), 1, g, a_d.cpu().numpy())
    parity.check_update(sub, g, 256, sums.cpu().numpy(), counts.cpu().numpy())
    # the trained codebooks quantise better than the synthetic Gaussian ones the other tests use
    codes = B.ivf_pq_encode(_t(x), _t(ids), _t(c), codebooks)
    rand_cb = _t(synth.pq_codebooks(pq_m, dsub, 0.3, seed=41))
    codes_r = B.ivf_pq_encode(_t(x), _t(ids), _t(c), rand_cb)
    def err(cb_t, cd):
        cbn, cdn = cb_t.cpu().numpy(), cd.cpu().numpy()
        dec = np.concatenate([cbn[m, cdn[:, m]] for m in range(pq_m)], axis=1)
        return ((want - dec) ** 2).sum(1).mean()
    assert err(codebooks, codes) < 0.8 * err(rand_cb, codes_r)


def test_codebook_training_with_sub_vectors_of_three():
    # DEEP-shaped width: 96 / 32 = 3 coordinates per subspace (padded to 4 inside the training helper)
    from paper_2608_08751_b200 import pq_train
    rng = np.random.default_rng(43)
    n, nlist, d, pq_m = 3000, 10, 24, 8
    c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
    ids, _ = synth.skewed_list_ids(n, nlist, seed=43)
    x = synth.rows_near(c, ids, 0.3, 43)
    codebooks, inertia = pq_train.train_codebooks(_t(x), _t(ids), _t(c), pq_m, iters=3, seed=2, method="assign")
    B.ivf_check()
    assert codebooks.shape == (pq_m, 256, 3) and torch.isfinite(codebooks).all()
    assert (np.diff(inertia.numpy(), axis=1) <= 1e-6 * inertia.numpy()[:, :-1]).all()
    want = O.pq_encode(x, ids, c, codebooks.cpu().numpy())
    got = B.ivf_pq_encode(_t(x), _t(ids), _t(c), codebooks.contiguous())
    B.ivf_check()
    assert (got.cpu().numpy() == want).all()


@pytest.mark.parametrize("d,pq_m", [(32, 8), (24, 8)])
def test_codebook_training_through_the_encoder(d, pq_m):
    # the default training method: assignment = the encoder over all subspaces, update = the sum/count
    # kernel with the code bytes as list ids.  Every iteration is checked against the oracle: the codes
    # it used (bit-identical) and the means it produced; the quantisation error never increases.
    from paper_2608_08751_b200 import pq_train
    rng = np.random.default_rng(47)
    n, nlist = 5000, 12
    dsub = d // pq_m
    c = rng.normal(0, 1, (nlist, d)).astype(np.float32)
    ids, _ = synth.skewed_list_ids(n, nlist, seed=47)
    x = synth.rows_near(c, ids, 0.3, 47)
    res = O.residuals(x, ids, c)

    def err(cb):
        codes = O.pq_encode(x, ids, c, cb)
        dec = np.concatenate([cb[m, codes[:, m]] for m in range(pq_m)], axis=1)
        return float(((res.astype(np.float64) - dec) ** 2).sum())

    prev_cb, prev_err = None, None
    for iters in (1, 2, 3):
        cb, inertia = pq_train.train_codebooks(_t(x), _t(ids), _t(c), pq_m, iters=iters, seed=5)
        B.ivf_check()
        cb = cb.cpu().numpy()
        assert inertia is None and cb.shape == (pq_m, 256, dsub)
        if prev_cb is not None:
            # one oracle Lloyd step from the previous codebooks reproduces this iteration
            codes = O.pq_encode(x, ids, c, prev_cb)
            for m in range(pq_m):
                sub = np.ascontiguousarray(res[:, m * dsub:(m + 1) * dsub])
                sums, counts, ok = O.update(sub, codes[:, m].astype(np.int32), 256)
                want = O.finalize(sums, counts, prev_cb[m])
                assert np.allclose(cb[m], want, rtol=2e-6, atol=1e-7)
        e = err(cb)
        assert prev_err is None or e <= prev_err * (1 + 1e-9)
        prev_cb, prev_err = cb, e
