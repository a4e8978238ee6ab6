"""How a routing result is compared with the CPU oracle's (spec tolerance).

TEST INFRASTRUCTURE ONLY, like the rest of this package: the tests assert on these figures and the
benchmark's CPU-baseline leg reports them.  Nothing here is reachable from the product path.

The rule.  tol(i, j) = 1e-3 * (|x_i|^2 + |c_j|^2) belongs to a (point, centroid) pair.
  * every returned distance lies within tol of the true (fp64, difference-form) distance;
  * membership at the k-th place: an oracle id whose distance is clearly below the oracle's k-th
    (by more than its tolerance) must be returned, and no returned id may lie clearly above it;
  * order inside the list ("chained" rule): no returned id's (true distance - tolerance) may exceed
    a later id's (true distance + tolerance).
The stricter position-by-position rule (where the two lists differ at a position, the two distances
at that position differ by less than the larger tolerance) is evaluated as well and reported, with
how far ids moved against the oracle's list, so that the effect of the chained rule is visible.
"""
from __future__ import annotations

import numpy as np

from . import oracle

REL_TOL = 1e-3


def route_agreement(xs: np.ndarray, c: np.ndarray, k: int, gpu_ids, gpu_dists=None, oracle_result=None) -> dict:
    """xs: the rows that were routed, c: centroids, gpu_ids [rows, k] (gpu_dists optional).
    Runs the oracle on xs (or takes its (ids, dists) for exactly these rows from `oracle_result`) and
    returns per-row boolean arrays and summary figures; asserts nothing."""
    gpu_ids = np.asarray(gpu_ids).reshape(-1, k).astype(np.int64)
    n, nlist = xs.shape[0], c.shape[0]
    if oracle_result is None:
        o_ids, o_d, _ = oracle.route(xs, c, k)
    else:
        o_ids, o_d = oracle_result
    xn, cn = oracle.sqnorms(xs), oracle.sqnorms(c)
    in_range = (gpu_ids >= 0) & (gpu_ids < nlist)
    safe = np.where(in_range, gpu_ids, 0)
    rr = np.repeat(np.arange(n, dtype=np.int64), k)
    Dg = oracle.pair_dists(xs, c, rr, safe.ravel()).reshape(n, k)  # true distance of each returned id
    tol_g = REL_TOL * (xn[:, None] + cn[safe])
    tol_o = REL_TOL * (xn[:, None] + cn[o_ids])
    dk = o_d[:, -1]
    must = o_d < (dk[:, None] - tol_o)
    # position of every returned id in the oracle's list (-1: not there), by sorting both lists
    pos_in_oracle = np.full((n, k), -1, np.int64)
    so = np.argsort(o_ids, axis=1, kind="stable")
    o_sorted = np.take_along_axis(o_ids, so, axis=1)
    for i in range(n):
        at = np.searchsorted(o_sorted[i], safe[i])
        at = np.minimum(at, k - 1)
        hit = o_sorted[i][at] == safe[i]
        pos_in_oracle[i, hit] = so[i][at[hit]]
    shared = pos_in_oracle >= 0
    present = np.zeros((n, k), bool)  # oracle position p is among the returned ids
    for i in range(n):
        present[i, pos_in_oracle[i][shared[i]]] = True
    member_ok = (present | ~must).all(axis=1) & (Dg <= dk[:, None] + tol_g).all(axis=1)
    lower = np.maximum.accumulate(Dg - tol_g, axis=1)
    chained_ok = (lower[:, :-1] <= (Dg + tol_g)[:, 1:]).all(axis=1) if k > 1 else np.ones(n, bool)
    differs = gpu_ids != o_ids
    gap = np.abs(Dg - o_d)
    positional_ok = ~(differs & ~(gap < np.maximum(tol_g, tol_o))).any(axis=1)
    disp = np.where(shared, np.abs(pos_in_oracle - np.arange(k)[None, :]), 0)
    out = {
        "rows": int(n), "o_ids": o_ids, "o_d": o_d, "true_d": Dg, "tol_g": tol_g, "in_range": in_range,
        "member_ok": member_ok, "chained_ok": chained_ok, "positional_ok": positional_ok,
        "rows_identical": float((~differs).all(axis=1).mean()),
        "positions_differing": int(differs.sum()),
        "top_k_set_overlap": float(shared.mean()),
        "max_displacement": int(disp.max()) if disp.size else 0,
        "ids_outside_oracle_list": int((~shared).sum()),
        "rows_passing_only_chained_rule": int((member_ok & chained_ok & ~positional_ok).sum()),
    }
    if gpu_dists is not None:
        gd = np.asarray(gpu_dists, dtype=np.float64).reshape(n, k)
        err = np.abs(gd - Dg)
        out["dist_ok"] = (err <= tol_g).all(axis=1)
        out["max_err_over_tol"] = float(np.max(err / tol_g)) if err.size else 0.0
    return out


def summary(a: dict) -> dict:
    """The JSON-friendly part of route_agreement's result."""
    ok = a["member_ok"] & a["chained_ok"] & a["in_range"].all(axis=1)
    if "dist_ok" in a:
        ok = ok & a["dist_ok"]
    out = {
        "rows_matching_oracle_by_tolerance_rule": float(ok.mean()),
        "rows_with_identical_id_lists": a["rows_identical"],
        "top_k_set_overlap": a["top_k_set_overlap"],
        "max_position_displacement": a["max_displacement"],
        "rows_passing_only_by_the_chained_order_rule": a["rows_passing_only_chained_rule"],
    }
    if "max_err_over_tol" in a:
        out["max_distance_error_over_tolerance"] = a["max_err_over_tol"]
    return out
