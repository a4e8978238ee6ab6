"""The allocation-free centroid update, through the C-ABI, against the regular entry point.

Some callers cannot allocate device memory when they call (a maintenance thread beside a serving
process whose pool already owns all free memory, a loop that cannot afford cudaMalloc's device-wide
synchronisation).  For them the library carries its update scratch inside its own image.  The
scratch is shared by all calls and keeps the previous call's contents, so this test makes two calls
in a row with different sizes and checks each against ivf_centroid_update on the same inputs; the
file name keeps it last in collection order, so a stale-scratch bug cannot hide behind earlier tests.
"""
import numpy as np
import pytest
import torch

from paper_2608_08751_b200 import binding as B

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
        code = B.IVF_U8 if x.dtype == np.uint8 else B.IVF_F32
        stream = torch.cuda.current_stream().cuda_stream
        rc = fn(xt.data_ptr(), code, it.data_ptr(), n, d, nlist, sums.data_ptr(), counts.data_ptr(), stream)
        assert rc == B.IVF_OK, B.lib().ivf_last_error().decode()
        torch.cuda.synchronize()
        out.append((sums.cpu().numpy(), counts.cpu().numpy()))
    return out


def _check(x, ids, nlist):
    (s_new, c_new), (s_ref, c_ref) = _both(x, ids, nlist)
    assert (c_new == c_ref).all() and c_new.sum() == x.shape[0]
    if x.dtype == np.uint8:
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
