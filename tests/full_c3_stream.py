"""The IVF-build configuration at full size with the CPU oracle beside it (not collected by pytest:
it streams 12.8 GB and takes minutes; run it by hand on a GPU machine):

    python tests/full_c3_stream.py [--n 100000000] [--iters 5] [--check-rows 10000]

Streams --n SIFT-shaped uint8 rows from page-locked host memory through --iters Lloyd iterations
(1,048,576-row chunks: assign k = 1, per-list sum/count update; then the finalize) with
``paper_2608_08751_b200.run_case.stream_case`` and, between iterations and outside the timing, lets
the oracle assign --check-rows seeded rows against the centroids that iteration used.  A GPU id
passes if its true distance is within the tolerance of the oracle's nearest distance and the
returned distance is within the tolerance of the true one (tolerance 1e-3 (|x|^2 + |c|^2)).
Prints one JSON line; exits non-zero if a check fails.
"""
import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import oracle  # noqa: E402
from paper_2608_08751_b200 import run_case  # noqa: E402


def checker(sample, c_now, g_ids, g_d):
    rows = sample.shape[0]
    g_d = g_d.astype(np.float64)
    o_ids, o_d = oracle.assign(sample, c_now)
    true_d = oracle.pair_dists(sample, c_now, np.arange(rows), g_ids)
    tol = 1e-3 * (oracle.sqnorms(sample) + oracle.sqnorms(c_now)[g_ids])
    ok = (true_d <= o_d + tol) & (np.abs(g_d - true_d) <= tol)
    return {"oracle_rows": int(rows), "rows_identical_to_oracle": float((g_ids == o_ids).mean()),
            "rows_within_tolerance_rule": float(ok.mean()),
            "max_distance_error_over_tolerance": float(np.max(np.abs(g_d - true_d) / tol))}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=100_000_000)
    ap.add_argument("--nlist", type=int, default=65_536)
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--check-rows", type=int, default=10_000, dest="check_rows")
    ap.add_argument("--dtype", default="u8")
    args = ap.parse_args()
    import contextlib
    import io
    buf = io.StringIO()
    with contextlib.redirect_stdout(buf):
        run_case.stream_case(args, checker=checker)
    line = json.loads(buf.getvalue().strip().splitlines()[-1])
    print(json.dumps(line))
    good = line["inertia_non_increasing"] and all(
        r["rows_within_tolerance_rule"] == 1.0 and r["counts_equal_bincount_of_all_ids"] and r["counts_total"] == args.n
        for r in line["iterations"])
    sys.exit(0 if good else 1)


if __name__ == "__main__":
    main()
