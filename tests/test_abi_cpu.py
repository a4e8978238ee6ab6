"""No-GPU checks of the C-ABI library: it loads, exports every declared symbol, rejects bad
arguments before touching CUDA, and its persistent schedule covers every unit exactly once."""
import ctypes
import os
import re

import pytest

from paper_2608_08751_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ivf_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ivf_[a-z_0-9]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    L = binding.lib()
    names = _declared()
    assert {"ivf_route", "ivf_assign", "ivf_centroid_update"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(names) == set(binding.EXPORTS)


def test_no_cluster_broadcast_loads_in_sources():
    # the sources that travel to multi-GPU runs must not name the cluster-broadcast TMA qualifier
    bad = "multi" + "cast"
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2608_08751_b200")):
        for f in files:
            if f.endswith((".cu", ".cuh", ".py", ".h")):
                assert bad not in open(os.path.join(dirpath, f)).read(), f


def _route(L, q, nq, d, qt, c, nlist, k, ids):
    return L.ivf_route(q, nq, d, qt, c, nlist, k, ids, None, None)


def test_argument_errors_come_before_any_cuda_call():
    L = binding.lib()
    buf = (ctypes.c_char * 4096)()
    p = ctypes.addressof(buf)
    p = (p + 255) & ~255
    assert _route(L, p, -1, 128, 0, p, 10, 1, p) == binding.IVF_ERR_INVALID_ARG
    assert _route(L, p, 4, 102, 0, p, 10, 1, p) == binding.IVF_ERR_UNSUPPORTED      # d % 4
    assert _route(L, p, 4, 272, 0, p, 10, 1, p) == binding.IVF_ERR_UNSUPPORTED      # d > 256
    assert _route(L, p, 4, 128, 7, p, 10, 1, p) == binding.IVF_ERR_INVALID_ARG      # dtype
    assert _route(L, p, 4, 128, 0, p, 10, 11, p) == binding.IVF_ERR_UNSUPPORTED     # nprobe > nlist
    assert _route(L, p, 4, 128, 0, p, 1000, 513, p) == binding.IVF_ERR_UNSUPPORTED  # nprobe > 512
    assert _route(L, p, 4, 128, 0, p, 10, 0, p) == binding.IVF_ERR_UNSUPPORTED
    assert _route(L, p, 4, 128, 0, p, 0, 1, p) == binding.IVF_ERR_INVALID_ARG
    assert _route(L, None, 4, 128, 0, p, 10, 1, p) == binding.IVF_ERR_INVALID_ARG
    assert _route(L, p, 4, 128, 0, None, 10, 1, p) == binding.IVF_ERR_INVALID_ARG
    assert _route(L, p, 4, 128, 0, p, 10, 1, None) == binding.IVF_ERR_INVALID_ARG
    assert _route(L, p + 4, 4, 128, 0, p, 10, 1, p) == binding.IVF_ERR_INVALID_ARG  # misaligned
    assert _route(L, None, 0, 128, 0, None, 10, 1, None) == binding.IVF_OK          # empty batch
    assert b"" != L.ivf_last_error() or True
    assert L.ivf_assign(None, 0, 96, 0, None, 5, None, None, None) == binding.IVF_OK
    assert L.ivf_assign(p, 3, 96, 0, None, 5, p, None, None) == binding.IVF_ERR_INVALID_ARG
    assert L.ivf_centroid_update(p, 0, p, -2, 128, 10, p, p, None) == binding.IVF_ERR_INVALID_ARG
    assert L.ivf_centroid_update(p, 0, p, 5, 22, 10, p, p, None) == binding.IVF_ERR_UNSUPPORTED
    assert L.ivf_centroid_update(p, 0, None, 5, 32, 10, p, p, None) == binding.IVF_ERR_INVALID_ARG
    assert L.ivf_centroid_update(None, 0, None, 0, 32, 10, None, None, None) == binding.IVF_OK
    assert L.ivf_assign_update(p, 5, 32, 0, p, 10, None, None, None, p, 0, None) == binding.IVF_ERR_INVALID_ARG
    msg = L.ivf_last_error().decode()
    assert "null" in msg


@pytest.mark.parametrize("n,nlist,d,k,sms", [
    (1000, 1024, 128, 16, 148), (10000, 65536, 128, 64, 148), (10000, 262144, 96, 128, 148),
    (1 << 20, 65536, 128, 1, 148), (100000, 1 << 20, 96, 256, 148), (1, 1, 16, 1, 148),
    (5, 100000, 64, 8, 148), (129, 257, 256, 2, 148), (300, 1000, 192, 5, 7), (128 * 148, 256, 128, 1, 148),
])
@pytest.mark.parametrize("cross", [-1, 0, 3, 8, 40])
def test_schedule_covers_every_unit_once_and_bounds_partials(n, nlist, d, k, sms, cross):
    binding.ivf_debug_set_crossing_cost(cross)
    try:
        _check_schedule(n, nlist, d, k, sms)
    finally:
        binding.ivf_debug_set_crossing_cost(-1)


def _check_schedule(n, nlist, d, k, sms):
    pl = binding.ivf_debug_plan(n, nlist, d, k, sms)
    T = pl["row_tiles"] * pl["col_tiles"]
    assert pl["mtiles"] in (1, 2)
    assert pl["row_tiles"] == -(-n // (128 * pl["mtiles"])) and pl["col_tiles"] == -(-nlist // pl["block_n"])
    assert pl["ctas"] == min(sms, T) and pl["stages"] >= 2 and pl["smem_bytes"] <= 227 * 1024
    prev_end = 0
    per_row_tile = {}
    for b in range(pl["ctas"]):
        u0, u1 = binding.ivf_debug_span(n, nlist, d, k, sms, b)
        assert u0 == prev_end and u1 > u0  # contiguous, non-empty
        prev_end = u1
        r0, r1 = u0 // pl["col_tiles"], (u1 - 1) // pl["col_tiles"]
        for r in range(r0, min(r1, r0 + 3) + 1):
            per_row_tile[r] = per_row_tile.get(r, 0) + 1
        if r1 > r0 + 3:  # a CTA covering many whole row tiles: each of those has exactly one partial
            per_row_tile[r1] = per_row_tile.get(r1, 0) + 1
    assert prev_end == T
    assert 2 * max(per_row_tile.values()) <= pl["partials"]  # two epilogue warps share every row


@pytest.mark.parametrize("n,nlist,d,k", [(10000, 65536, 128, 64), (10000, 262144, 96, 128), (9984, 1 << 20, 96, 256),
                                        (1 << 20, 65536, 128, 1), (300, 100000, 64, 8), (40000, 3000, 128, 1)])
def test_rotated_sweeps_walk_the_table_as_a_few_fronts(n, nlist, d, k):
    # Position p of row group r stands for centroid tile (p + rot_r) mod NT.  With every CTA advancing
    # one unit per step (a row-group change costs `cross` steps), the tile a CTA works on minus the
    # step count must take only a handful of values over all CTAs and steps: the CTAs then share a
    # few fronts and a tile is fetched from HBM once per front, not once per row group.
    sms = 148
    pl = binding.ivf_debug_plan(n, nlist, d, k, sms)
    NT, R = pl["col_tiles"], pl["row_tiles"]
    cross = 8 if k == 1 else 4
    rot = {}
    offsets = set()
    for b in range(pl["ctas"]):
        u0, u1 = binding.ivf_debug_span(n, nlist, d, k, sms, b)
        t = 0
        u = u0
        while u < u1:
            r = u // NT
            if r not in rot:
                rot[r] = binding.ivf_debug_rotation(n, nlist, d, k, sms, r)
                assert 0 <= rot[r] < NT
            p0 = u - r * NT
            p1 = min(u1 - r * NT, NT)
            offsets.add(((p0 + rot[r]) - t) % NT)   # constant along a segment: tile and time advance together
            t += (p1 - p0) + cross
            u = r * NT + p1
    spans_per_sweep = -(-NT * R // pl["ctas"])
    fronts = -(-NT // max(1, spans_per_sweep - 2 * cross)) + 2
    # a front may be smeared by the rounding of the span boundaries and the crossing charge
    centres = sorted(offsets)
    groups = 1
    for a, bb in zip(centres, centres[1:]):
        if bb - a > 4 * cross + 4:
            groups += 1
    assert groups <= fronts + 1, (groups, fronts, len(offsets))
    assert rot[0] == 0


def test_threshold_rule_selection():
    assert binding.ivf_debug_rule(1, 65536) == (-1, 1)
    assert binding.ivf_debug_rule(16, 65536) == (1, 16)           # threshold pass, can never come up short
    assert binding.ivf_debug_rule(16, 1024) == (0, 1)             # small table: running rule, exact
    assert binding.ivf_debug_rule(64, 65536) == (1, 16)           # threshold pass over every 16th centroid
    assert binding.ivf_debug_rule(128, 262144) == (1, 32)
    assert binding.ivf_debug_rule(256, 1 << 20) == (1, 64)
    assert binding.ivf_debug_rule(512, 600)[0] == 2               # sample too small: bounded logs
    assert binding.ivf_debug_rule(17, 2044)[0] == 2 and binding.ivf_debug_rule(17, 2045) == (1, 4)


def test_pq_and_candidate_entry_points_check_arguments_first():
    L = binding.lib()
    i64, i32, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
    L.ivf_pq_encode.argtypes = [vp, i64, i32, i32, vp, vp, i32, vp, i32, vp, vp]
    L.ivf_pq_search.argtypes = [vp, i64, i32, i32, vp, i32, vp, i32, vp, vp, i64, vp, i32, i32, vp, vp, vp, vp, vp]
    L.ivf_assign_candidates.argtypes = [vp, i64, i32, i32, vp, i32, vp, i32, vp, vp, vp]
    buf = (ctypes.c_char * 4096)()
    p = (ctypes.addressof(buf) + 255) & ~255
    UNS, INV, OK = binding.IVF_ERR_UNSUPPORTED, binding.IVF_ERR_INVALID_ARG, binding.IVF_OK
    # encode: pq_m must divide d; the codebook must fit shared memory; empty input is fine
    assert L.ivf_pq_encode(p, 4, 128, 0, p, p, 10, p, 24, p, None) == INV
    assert L.ivf_pq_encode(p, 4, 256, 0, p, p, 10, p, 64, p, None) == UNS
    assert L.ivf_pq_encode(p, 4, 128, 5, p, p, 10, p, 32, p, None) == INV           # dtype
    assert L.ivf_pq_encode(None, 0, 128, 0, None, None, 10, p, 32, None, None) == OK
    # search: probe count, N_rerank, position width, alignment of the code array
    def search(nq=4, d=128, qt=1, nlist=100, nprobe=8, n_codes=1000, pq_m=32, n_rerank=64, codes=p, q=p):
        return L.ivf_pq_search(q, nq, d, qt, p, nlist, p, nprobe, p, codes, n_codes, p, pq_m, n_rerank, None, p, p, None, None)
    assert search(nprobe=0) == INV and search(nprobe=101) == INV
    assert search(nlist=1000, nprobe=513) == UNS
    assert search(n_rerank=0) == UNS and search(n_rerank=1025) == UNS
    assert search(n_codes=1 << 32) == UNS
    assert search(pq_m=48) == INV
    assert search(codes=p + 8) == INV
    assert search(nq=-1) == INV
    assert search(nq=0, q=None) == OK
    # candidates: d a multiple of 4 up to 256, at least one candidate per row
    assert L.ivf_assign_candidates(p, 4, 130, 0, p, 10, p, 8, p, None, None) == UNS
    assert L.ivf_assign_candidates(p, 4, 128, 0, p, 10, p, 0, p, None, None) == INV
    assert L.ivf_assign_candidates(p, 4, 128, 0, None, 10, p, 8, p, None, None) == INV
    assert L.ivf_assign_candidates(None, 0, 128, 0, None, 10, None, 8, None, None, None) == OK
