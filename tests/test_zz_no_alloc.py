"""The allocation-free centroid update, through the C-ABI, against the regular entry point.

Some callers cannot allocate device memory when they call (a maintenance thread beside a serving
process whose pool already owns all free memory, a loop that cannot afford cudaMalloc's device-wide
synchronisation).  For them the library carries its update scratch inside its own image.  The
scratch is shared by all calls and keeps the previous call's contents, so this test makes two calls
in a row with different sizes and checks each against ivf_centroid_update on the same inputs and
against the CPU oracle; the file name keeps it last in collection order, so a stale-scratch bug
cannot hide behind earlier tests.  Further cases: the largest sizes the built-in scratch takes,
signed-byte rows, accumulation on top of sums and counts that are already there, and ids out of
range (skipped, and -- unlike the regular entry point -- not reported through ivf_check).
"""
import numpy as np
import pytest
import torch

from paper_2608_08751_b200 import binding as B

import parity

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _both(x, ids, nlist):
    """(sums, counts) from the allocation-free entry point and from the regular one."""
    n, d = x.shape
    xt, it = _cuda(x), _cuda(ids)
    out = []
    for fn in (B.lib().ivf_centroid_update_noalloc, B.lib().ivf_centroid_update):
        sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
        counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
        code = {np.dtype(np.uint8): B.IVF_U8, np.dtype(np.int8): B.IVF_I8}.get(x.dtype, B.IVF_F32)
        stream = torch.cuda.current_stream().cuda_stream
        rc = fn(xt.data_ptr(), code, it.data_ptr(), n, d, nlist, sums.data_ptr(), counts.data_ptr(), stream)
        assert rc == B.IVF_OK, B.lib().ivf_last_error().decode()
        torch.cuda.synchronize()
        out.append((sums.cpu().numpy(), counts.cpu().numpy()))
    return out


def _check(x, ids, nlist):
    (s_new, c_new), (s_ref, c_ref) = _both(x, ids, nlist)
    assert (c_new == c_ref).all() and c_new.sum() == x.shape[0]
    parity.check_update(x, ids, nlist, s_new, c_new)  # the oracle: counts bit-exact, sums exact / 1e-5 relative
    if x.dtype in (np.uint8, np.int8):
        assert (s_new == s_ref).all()  # integer sums below 2^24: exact in both
    else:
        mag = np.zeros_like(s_ref, dtype=np.float64)
        np.add.at(mag, ids, np.abs(x.astype(np.float64)))
        assert (np.abs(s_new.astype(np.float64) - s_ref) <= 1e-5 * mag + 1e-30).all()


def test_two_calls_in_a_row_match_the_regular_entry_point():
    rng = np.random.default_rng(21)
    # call 1: many lists, uint8 rows
    x1 = rng.integers(0, 256, (50_000, 128)).astype(np.uint8)
    ids1 = rng.integers(0, 65_536, 50_000).astype(np.int32)
    _check(x1, ids1, 65_536)
    # call 2: fewer rows and lists, float rows -- whatever call 1 left in the scratch must not matter
    x2 = rng.standard_normal((7_001, 96)).astype(np.float32)
    ids2 = rng.integers(0, 300, 7_001).astype(np.int32)
    _check(x2, ids2, 300)
    # and a third one: a prefix of the first rows folded into 50 lists
    _check(x1[:1000], ids1[:1000] % 50, 50)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    L = B.lib()
    x = torch.zeros((16, 32), dtype=torch.float32, device="cuda")
    ids = torch.zeros((16,), dtype=torch.int32, device="cuda")
    sums = torch.zeros((4, 32), dtype=torch.float32, device="cuda")
    counts = torch.zeros((4,), dtype=torch.int64, device="cuda")
    rc = L.ivf_centroid_update_noalloc(x.data_ptr(), 0, ids.data_ptr(), (1 << 20) + 1, 32, 4, sums.data_ptr(),
                                       counts.data_ptr(), None)
    assert rc == B.IVF_ERR_UNSUPPORTED and "1048576" in L.ivf_last_error().decode()
    rc = L.ivf_centroid_update_noalloc(x.data_ptr(), 0, ids.data_ptr(), 16, 32, 65_537, sums.data_ptr(),
                                       counts.data_ptr(), None)
    assert rc == B.IVF_ERR_UNSUPPORTED and "65536" in L.ivf_last_error().decode()
    torch.cuda.synchronize()
    assert counts.sum().item() == 0  # nothing ran


def _noalloc(x, ids, nlist, sums, counts):
    code = {np.dtype(np.uint8): B.IVF_U8, np.dtype(np.int8): B.IVF_I8}.get(x.dtype, B.IVF_F32)
    xt, it = _cuda(x), _cuda(ids)
    rc = B.lib().ivf_centroid_update_noalloc(xt.data_ptr(), code, it.data_ptr(), x.shape[0], x.shape[1], nlist,
                                             sums.data_ptr(), counts.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == B.IVF_OK, B.lib().ivf_last_error().decode()
    torch.cuda.synchronize()


def test_largest_sizes_the_built_in_scratch_takes():
    # n = 1,048,576 rows into 65,536 lists: the last element of the permutation and the last offset slot
    n, nlist, d = 1 << 20, 65_536, 128
    rng = np.random.default_rng(22)
    x = rng.integers(0, 256, (n, d), dtype=np.uint8)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    ids[-1] = nlist - 1
    ids[0] = 0
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    _noalloc(x, ids, nlist, sums, counts)
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy())
    # a small call right after the largest one: the scratch is full of the big call's leftovers
    x2 = rng.integers(0, 256, (333, 64), dtype=np.uint8)
    ids2 = rng.integers(0, 9, 333).astype(np.int32)
    sums2 = torch.zeros((9, 64), dtype=torch.float32, device="cuda")
    counts2 = torch.zeros((9,), dtype=torch.int64, device="cuda")
    _noalloc(x2, ids2, 9, sums2, counts2)
    parity.check_update(x2, ids2, 9, sums2.cpu().numpy(), counts2.cpu().numpy())


@pytest.mark.parametrize("dtype,d", [(np.int8, 100), (np.float32, 36)])
def test_signed_bytes_and_accumulation_on_existing_sums(dtype, d):
    n, nlist = 20_000, 777
    rng = np.random.default_rng(23)
    if dtype == np.int8:
        x = rng.integers(-128, 128, (n, d)).astype(np.int8)
    else:
        x = rng.standard_normal((n, d)).astype(np.float32)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    ids[ids == 5] = 6  # an empty list keeps what it had
    base_s = rng.integers(-50, 50, (nlist, d)).astype(np.float32)
    base_c = rng.integers(0, 1000, nlist).astype(np.int64)
    sums, counts = _cuda(base_s.copy()), _cuda(base_c.copy())
    h = n // 3
    _noalloc(x[:h], ids[:h], nlist, sums, counts)
    _noalloc(x[h:], ids[h:], nlist, sums, counts)
    parity.check_update(x, ids, nlist, sums.cpu().numpy(), counts.cpu().numpy(), base_s.astype(np.float64), base_c)
    assert (sums.cpu().numpy()[5] == base_s[5]).all() and counts.cpu().numpy()[5] == base_c[5]


def test_ids_out_of_range_are_skipped_and_not_reported():
    n, nlist, d = 5_000, 40, 32
    rng = np.random.default_rng(24)
    x = rng.integers(0, 256, (n, d), dtype=np.uint8)
    ids = rng.integers(0, nlist, n).astype(np.int32)
    bad = rng.choice(n, 60, replace=False)
    ids[bad[:30]] = -7
    ids[bad[30:]] = nlist + 3
    sums = torch.zeros((nlist, d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((nlist,), dtype=torch.int64, device="cuda")
    _noalloc(x, ids, nlist, sums, counts)
    good = (ids >= 0) & (ids < nlist)
    parity.check_update(x[good], ids[good], nlist, sums.cpu().numpy(), counts.cpu().numpy())
    assert counts.sum().item() == n - 60
    B.ivf_check()  # this variant leaves the library's status word alone
