"""The comparison rule itself (oracle/compare.py) on hand-made lists: what it accepts, what it
rejects, and the displacement figures it reports."""
import numpy as np

from oracle import compare, oracle


def _case():
    # one 1-D query at 100 (|x|^2 = 1e4) and centroids at 100 + offsets: distance = offset^2.
    # tolerance of a pair = 1e-3 * (1e4 + c^2) ~ 20..25
    offs = np.array([1.0, 2.0, 2.05, 9.0, 9.2, 30.0, 31.0, 60.0], np.float64)
    c = np.zeros((8, 4), np.float32)
    c[:, 0] = (100.0 + offs).astype(np.float32)
    x = np.zeros((1, 4), np.float32)
    x[0, 0] = 100.0
    return x, c


def test_identical_lists_and_reported_figures():
    x, c = _case()
    ids, d, _ = oracle.route(x, c, 5)
    assert ids[0].tolist() == [0, 1, 2, 3, 4]
    a = compare.route_agreement(x, c, 5, ids, d)
    s = compare.summary(a)
    assert s["rows_matching_oracle_by_tolerance_rule"] == 1.0 and s["rows_with_identical_id_lists"] == 1.0
    assert s["max_position_displacement"] == 0 and s["rows_passing_only_by_the_chained_order_rule"] == 0


def test_swap_inside_the_tolerance_passes_and_is_counted():
    x, c = _case()
    ids = np.array([[0, 2, 1, 4, 3]], np.int32)  # 4 vs 4.2 and 81 vs 84.6: both gaps inside ~20
    d = oracle.pair_dists(x, c, np.zeros(5, np.int64), ids[0]).reshape(1, 5)
    a = compare.route_agreement(x, c, 5, ids, np.sort(d, axis=1))
    assert a["member_ok"].all() and a["chained_ok"].all() and a["positional_ok"].all()
    assert a["max_displacement"] == 1 and a["positions_differing"] == 4


def test_swap_beyond_the_tolerance_fails_the_order_rule():
    x, c = _case()
    ids = np.array([[0, 1, 3, 2, 4]], np.int32)  # 81 before 4.2: gap 77 > 2 tolerances
    a = compare.route_agreement(x, c, 5, ids)
    assert a["member_ok"].all() and not a["chained_ok"].any() and not a["positional_ok"].any()


def test_missing_clear_member_and_clear_outsider_fail_membership():
    x, c = _case()
    ids = np.array([[0, 1, 2, 3, 5]], np.int32)  # 900 returned instead of 84.6
    a = compare.route_agreement(x, c, 5, ids)
    assert not a["member_ok"].any()
    assert a["ids_outside_oracle_list"] == 1
    ids = np.array([[1, 2, 3, 4, 5]], np.int32)  # the nearest centroid (1 vs k-th 84.6) is missing
    a = compare.route_agreement(x, c, 5, ids)
    assert not a["member_ok"].any()


def test_boundary_swap_inside_the_tolerance_is_accepted():
    x, c = _case()
    ids = np.array([[0, 1, 2, 4]], np.int32)  # k = 4: 84.6 instead of 81 at the k-th place
    a = compare.route_agreement(x, c, 4, ids)
    assert a["member_ok"].all() and a["chained_ok"].all()
    assert a["top_k_set_overlap"] == 0.75
