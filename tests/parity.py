"""Comparison of the CUDA path's results with the CPU oracle's, by the stated rule:
distances within 1e-3 * (|x|^2 + |c|^2); id lists equal to the oracle's except where the true
distances of the ids involved lie within that tolerance of each other (membership at the k-th
place, order inside the list)."""
import numpy as np

from oracle import compare, oracle

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
    a = compare.route_agreement(xs, c, k, gpu_ids, gpu_dists)

    assert a["in_range"].all(), "id out of range"
    srt = np.sort(gpu_ids, axis=1)
    assert (srt[:, 1:] != srt[:, :-1]).all(), "duplicate id in a row"
    assert (np.diff(gpu_dists, axis=1) >= 0).all(), "row not ascending in its own distances"
    assert a["dist_ok"].all(), f"distance off by {a['max_err_over_tol']:.3g} x tolerance"
    if exact:
        assert (gpu_ids == a["o_ids"]).all(), "ids differ on an integer-exact case"
        assert (gpu_dists == a["o_d"]).all(), "distances differ on an integer-exact case"
    # membership at the k-th place, then the order inside the list: every returned id carries its own
    # tolerance (it grows with |c|^2), so an id may sit later than a truly farther one only if the two
    # true distances can be reconciled within their tolerances
    assert a["member_ok"].all(), "an id clearly inside the top-k is missing, or one clearly outside was returned"
    assert a["chained_ok"].all(), "order differs beyond the tolerance"
    return {
        "rows": a["rows"],
        "rows_identical": a["rows_identical"],
        "positions_differing": a["positions_differing"],
        "max_err_over_tol": a["max_err_over_tol"],
        "max_displacement": a["max_displacement"],
        "rows_passing_only_chained_rule": a["rows_passing_only_chained_rule"],
    }


def check_all_row_distances(x, c, k, gpu_ids, gpu_dists):
    """Every returned (row, id) pair re-checked against the definition (n * k * d work in fp64,
    independent of the full oracle): distance within tolerance, ids in range and distinct, rows
    ascending.  Holds at any size."""
    n, nlist = x.shape[0], c.shape[0]
    gpu_ids = np.asarray(gpu_ids).reshape(n, k)
    gpu_dists = np.asarray(gpu_dists).reshape(n, k)
    assert ((gpu_ids >= 0) & (gpu_ids < nlist)).all(), "id out of range"
    if k > 1:
        s = np.sort(gpu_ids, axis=1)
        assert (s[:, 1:] != s[:, :-1]).all(), "duplicate id in a row"
        assert (np.diff(gpu_dists, axis=1) >= 0).all(), "row not ascending in its own distances"
    xn, cn = oracle.sqnorms(x), oracle.sqnorms(c)
    worst = 0.0
    step = max(1, (1 << 24) // k)
    for r0 in range(0, n, step):  # bounded temporaries
        r1 = min(n, r0 + step)
        rr = np.repeat(np.arange(r0, r1, dtype=np.int64), k)
        ids = gpu_ids[r0:r1].ravel().astype(np.int64)
        D = oracle.pair_dists(x, c, rr, ids)
        tol = REL_TOL * (xn[rr] + cn[ids])
        err = np.abs(gpu_dists[r0:r1].ravel().astype(np.float64) - D)
        assert (err <= tol).all(), f"distance off by {np.max(err / tol):.3g} x tolerance"
        worst = max(worst, float(np.max(err / tol)))
    return worst


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
