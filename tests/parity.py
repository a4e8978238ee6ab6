"""Comparison of the CUDA path's results with the CPU oracle's, by the stated rule:
distances within 1e-3 * (|x|^2 + |c|^2); id lists equal to the oracle's except where the true
distances of the ids involved lie within that tolerance of each other (membership at the k-th
place, order inside the list)."""
import numpy as np

from oracle import oracle

REL_TOL = 1e-3


def check_route(x, c, k, gpu_ids, gpu_dists, rows=None, exact=False):
    """x: all points (numpy), c: centroids; gpu_ids/gpu_dists: [len(rows), k] results for `rows`
    (default: all rows).  Runs the oracle on those rows.  Returns statistics; raises on mismatch."""
    gpu_ids = np.asarray(gpu_ids).reshape(-1, k)
    gpu_dists = np.asarray(gpu_dists, dtype=np.float64).reshape(-1, k)
    if rows is None:
        rows = np.arange(x.shape[0])
    rows = np.asarray(rows, np.int64)
    xs = np.ascontiguousarray(x[rows])
    n, nlist = xs.shape[0], c.shape[0]
    o_ids, o_d, o_next = oracle.route(xs, c, k)
    xn = oracle.sqnorms(xs)
    cn = oracle.sqnorms(c)

    assert ((gpu_ids >= 0) & (gpu_ids < nlist)).all(), "id out of range"
    srt = np.sort(gpu_ids, axis=1)
    assert (srt[:, 1:] != srt[:, :-1]).all(), "duplicate id in a row"
    assert (np.diff(gpu_dists, axis=1) >= 0).all(), "row not ascending in its own distances"

    rr = np.repeat(np.arange(n, dtype=np.int64), k)
    Dg = oracle.pair_dists(xs, c, rr, gpu_ids.ravel()).reshape(n, k)  # true distance of each returned id
    tol_g = REL_TOL * (xn[:, None] + cn[gpu_ids])
    err = np.abs(gpu_dists - Dg)
    assert (err <= tol_g).all(), f"distance off by {np.max(err / tol_g):.3g} x tolerance"

    if exact:
        assert (gpu_ids == o_ids).all(), "ids differ on an integer-exact case"
        assert (gpu_dists == o_d).all(), "distances differ on an integer-exact case"

    tol_o = REL_TOL * (xn[:, None] + cn[o_ids])
    dk = o_d[:, -1]
    must = o_d < (dk[:, None] - tol_o)
    present = (o_ids[:, :, None] == gpu_ids[:, None, :]).any(-1)
    assert (present | ~must).all(), "an id clearly inside the top-k is missing"
    assert (Dg <= dk[:, None] + tol_g).all(), "an id clearly outside the top-k was returned"
    # Order inside the list.  Every returned id carries its own tolerance (it grows with |c|^2), so an
    # id may sit later than a truly farther one only if the two true distances can be reconciled
    # within their tolerances: no id's (true distance - tolerance) may exceed a later id's (true
    # distance + tolerance).  (Comparing position by position with the oracle's list is stricter than
    # the stated tolerance: one id displaced within its own, larger, tolerance shifts the ids between.)
    lower = np.maximum.accumulate(Dg - tol_g, axis=1)
    assert (lower[:, :-1] <= (Dg + tol_g)[:, 1:]).all(), "order differs beyond the tolerance"
    differs = gpu_ids != o_ids
    return {
        "rows": int(n),
        "rows_identical": float((~differs).all(axis=1).mean()),
        "positions_differing": int(differs.sum()),
        "max_err_over_tol": float(np.max(err / tol_g)),
    }


def check_update(x, ids, nlist, gpu_sums, gpu_counts, base_sums=None, base_counts=None):
    """counts bit-exact; sums within 1e-5 * sum_i |x_it| over the members (exact for uint8)."""
    sums, counts, ok = oracle.update(x, ids, nlist)
    assert ok
    if base_counts is not None:
        counts = counts + base_counts
        sums = sums + base_sums
    assert (np.asarray(gpu_counts) == counts).all(), "counts differ"
    gs = np.asarray(gpu_sums, dtype=np.float64)
    if x.dtype in (np.uint8, np.int8) and np.abs(sums).max() < 2 ** 24:
        assert (gs == sums).all(), "byte-typed sums must be exact"
        return 0.0
    mag = np.zeros_like(sums)
    np.add.at(mag, ids, np.abs(x.astype(np.float64)))
    if base_sums is not None:
        mag = mag + np.abs(base_sums)
    bound = 1e-5 * mag + 1e-30
    rel = np.abs(gs - sums) / bound
    assert (rel <= 1.0).all(), f"sums off by {rel.max():.3g} x tolerance"
    return float(rel.max())
