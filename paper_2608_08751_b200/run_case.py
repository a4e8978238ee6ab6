"""Runs one call of the library on seeded synthetic input of a chosen size and prints its timing.

A small driver for profilers and quick measurements:
    python -m paper_2608_08751_b200.run_case --op assign --n 262144 --nlist 65536 --d 128 --dtype u8 --reps 3
    python -m paper_2608_08751_b200.run_case --op route --n 10000 --nlist 65536 --k 64
    python -m paper_2608_08751_b200.run_case --op update --n 1048576 --nlist 65536
    python -m paper_2608_08751_b200.run_case --op stream --n 8388608 --nlist 65536 --iters 2
    python -m paper_2608_08751_b200.run_case --op serve --nlist 524288 --k 64 --batches 8,32,256,2048
"serve" routes small query batches against a prepared, device-resident centroid table (the paper's
serving setting: N_list = 0.5M, batch sizes 8 to 2048) and reports the time per batch.
"stream" is the IVF-build configuration in small: rows in page-locked host memory, streamed in
1,048,576-row chunks through assign + update, then the finalize, per Lloyd iteration.
Inputs follow the SIFT-shaped (uint8, all-positive mixture) or DEEP-shaped (float32, unit norm)
recipes of ``synth``.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import synth


def _fill_chunks(host, args):
    """Seeded rows into the page-locked buffer, chunk by chunk (the recipe of the full configuration);
    numpy's generators release the interpreter lock, so a thread pool spreads the chunks over the cores."""
    from concurrent.futures import ThreadPoolExecutor
    import os
    chunk = synth.CHUNK_ROWS
    nchunks = -(-args.n // chunk)
    view = host.numpy()

    def fill(c):
        rows = min(chunk, args.n - c * chunk)
        if args.dtype == "u8":
            view[c * chunk:c * chunk + rows] = synth.sift_like_rows(c, rows=rows, d=args.d)
        else:
            view[c * chunk:c * chunk + rows] = synth.deep_like_rows(c, rows=rows, d=args.d)

    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as pool:
        list(pool.map(fill, range(nchunks)))
    return nchunks


def stream_case(args, checker=None):
    """The IVF-build configuration: rows in page-locked host memory, streamed in 1,048,576-row chunks
    through assign + update, then the finalize, per Lloyd iteration.  Every iteration is timed on its
    own with CUDA events.  `checker`, if given, is called between iterations (outside the timing) as
    checker(sample_rows, centroids_used, ids_of_sample, dists_of_sample) -> dict on --check-rows seeded
    rows; what it returns is added to the iteration's record (the test tree passes a checker that
    re-assigns the rows on the CPU).  The per-list counts are compared with a bincount of all ids."""
    import time
    t_gen = time.perf_counter()
    host = torch.empty((args.n, args.d), dtype=torch.uint8 if args.dtype == "u8" else torch.float32).pin_memory()
    nchunks = _fill_chunks(host, args)
    t_gen = time.perf_counter() - t_gen
    init = synth.init_sample(args.n, args.nlist)
    cent = host[torch.from_numpy(init)].to(torch.float32).cuda()
    sums = torch.zeros((args.nlist, args.d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((args.nlist,), dtype=torch.int64, device="cuda")
    ids = torch.empty((args.n,), dtype=torch.int32, device="cuda")
    dists = torch.empty((args.n,), dtype=torch.float32, device="cuda")

    def iteration():
        sums.zero_()
        counts.zero_()
        B.ivf_assign_update(host, cent, sums, counts, ids, dists)
        B.ivf_centroid_finalize(sums, counts, cent)

    # warm-up on a few chunks (workspace growth), on a copy of the centroids
    keep = cent.clone()
    sums.zero_()
    counts.zero_()
    B.ivf_assign_update(host[:min(args.n, 4 * synth.CHUNK_ROWS)], cent, sums, counts, ids, dists)
    B.ivf_check()
    cent.copy_(keep)
    check_rows = min(args.check_rows, args.n) if checker is not None else 0
    sel = np.sort(np.random.default_rng(33).choice(args.n, check_rows, replace=False)) if check_rows else None
    sample = np.ascontiguousarray(host.numpy()[sel]) if check_rows else None
    per_iter = []
    for it in range(args.iters):
        c_now = cent.cpu().numpy().copy() if check_rows else None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        iteration()
        e1.record()
        B.ivf_check()
        ms = e0.elapsed_time(e1)
        esize = 1 if args.dtype == "u8" else 4
        rec = {"iteration": it, "ms": ms, "vectors_per_s": args.n / (ms / 1e3),
               "host_link_GBps": args.n * args.d * esize / (ms / 1e3) / 1e9,
               "tflops": 2.0 * args.n * args.nlist * args.d / (ms / 1e3) / 1e12,
               "inertia": float(dists.double().sum().item()),
               "counts_total": int(counts.sum().item()), "empty_lists": int((counts == 0).sum().item())}
        if check_rows:
            at = torch.from_numpy(sel).cuda()
            rec.update(checker(sample, c_now, ids[at].cpu().numpy(), dists[at].cpu().numpy()))
        rec["counts_equal_bincount_of_all_ids"] = bool(
            (np.bincount(ids.cpu().numpy(), minlength=args.nlist) == counts.cpu().numpy()).all())
        per_iter.append(rec)
    total_ms = sum(r["ms"] for r in per_iter)
    inertia = [r["inertia"] for r in per_iter]
    print(json.dumps({"op": "stream", "n": args.n, "nlist": args.nlist, "d": args.d, "dtype": args.dtype,
                      "chunks": nchunks, "iterations": per_iter, "total_ms": total_ms,
                      "ms_per_iteration": total_ms / args.iters, "vectors_per_s": args.n * args.iters / (total_ms / 1e3),
                      "host_link_GBps": args.n * args.d * (1 if args.dtype == "u8" else 4) * args.iters / (total_ms / 1e3) / 1e9,
                      "tflops": 2.0 * args.n * args.nlist * args.d * args.iters / (total_ms / 1e3) / 1e12,
                      "inertia": inertia,
                      "inertia_non_increasing": all(b <= a * (1 + 1e-6) for a, b in zip(inertia, inertia[1:])),
                      "host_generation_s": t_gen}))


def build_case(args):
    """Index construction in the accelerated style (appendix on fast index building): the centroids
    are trained by Lloyd iterations on a SAMPLE of the base set (--train-rows), then every base
    vector is assigned once, regrouped list-major and residual-encoded.  Assignment is exact brute
    force here (no graph); everything streams from page-locked host memory."""
    chunk = synth.CHUNK_ROWS
    nchunks = -(-args.n // chunk)
    host = torch.empty((args.n, args.d), dtype=torch.uint8 if args.dtype == "u8" else torch.float32).pin_memory()
    _fill_chunks(host, args)
    train_rows = min(args.train_rows, args.n)
    train = host[:train_rows]
    init = synth.init_sample(train_rows, args.nlist)
    cent = train[torch.from_numpy(init)].to(torch.float32).cuda()
    sums = torch.zeros((args.nlist, args.d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((args.nlist,), dtype=torch.int64, device="cuda")
    ids = torch.empty((args.n,), dtype=torch.int32, device="cuda")
    B.ivf_assign_update(train[:4096], cent, sums, counts, None, None)  # warm-up (workspace growth)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    ev[0].record()
    for _ in range(args.iters):
        sums.zero_()
        counts.zero_()
        B.ivf_assign_update(train, cent, sums, counts, None, None)
        B.ivf_centroid_finalize(sums, counts, cent)
    ev[1].record()
    B.ivf_assign(host, cent, ids, None, want_dists=False)
    ev[2].record()
    dev_rows = host.cuda()
    xr, offsets, order = B.ivf_cluster_major_reorder(dev_rows, ids, args.nlist)
    ids_sorted = ids[order.long()]
    ev.append(torch.cuda.Event(enable_timing=True))
    ev[3].record()
    from . import pq_train
    cb, _ = pq_train.train_codebooks(xr, ids_sorted, cent, args.pq_m, iters=args.iters, seed=1,
                                     sample_rows=min(args.n, 1 << 20))
    ev.append(torch.cuda.Event(enable_timing=True))
    ev[4].record()
    codes = B.ivf_pq_encode(xr, ids_sorted, cent, cb)
    ev.append(torch.cuda.Event(enable_timing=True))
    ev[5].record()
    B.ivf_check()
    t = [ev[i].elapsed_time(ev[i + 1]) for i in range(5)]
    lens = (offsets[1:] - offsets[:-1])
    print(json.dumps({"op": "build", "n": args.n, "train_rows": train_rows, "nlist": args.nlist, "d": args.d,
                      "dtype": args.dtype, "iters": args.iters, "train_ms": t[0], "assign_all_ms": t[1],
                      "copy_reorder_ms": t[2], "pq_train_ms": t[3], "pq_encode_ms": t[4], "total_ms": sum(t),
                      "vectors_per_s": args.n / (sum(t) / 1e3),
                      "empty_lists": int((lens == 0).sum().item()), "max_list": int(lens.max().item()),
                      "codes_bytes": int(codes.numel())}))


def serve_case(args):
    if args.dtype == "u8":
        c = synth.sift_like_centroids(args.nlist, args.d)
        q_all = synth.sift_like_queries(max(int(v) for v in args.batches.split(",")), args.d)
    else:
        c = synth.deep_like_centroids(args.nlist, args.d)
        q_all = synth.deep_like_queries(max(int(v) for v in args.batches.split(",")), args.d)
    ct = torch.from_numpy(c).cuda()
    handle = B.PreparedCentroids(ct)
    out = {"op": "serve", "nlist": args.nlist, "d": args.d, "k": args.k, "dtype": args.dtype, "batches": {}}
    for bs in [int(v) for v in args.batches.split(",")]:
        q = torch.from_numpy(q_all[:bs]).cuda()
        ids = torch.empty((bs, args.k), dtype=torch.int32, device="cuda")
        dists = torch.empty((bs, args.k), dtype=torch.float32, device="cuda")
        for _ in range(3):
            B.ivf_route_prepared(handle, q, args.k, ids, dists)
        B.ivf_check()
        reps = max(args.reps, 20)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            B.ivf_route_prepared(handle, q, args.k, ids, dists)
        e1.record()
        B.ivf_check()
        us = e0.elapsed_time(e1) / reps * 1e3
        out["batches"][str(bs)] = {"us_per_batch": us, "queries_per_s": bs / (us / 1e6)}
    handle.close()
    print(json.dumps(out))


def pq_case(args):
    """The PQ pipeline on the library's own calls: assign -> list-major reorder -> residual encoding
    (timed once), then per batch: routing (prepared table) -> candidate reduction (timed)."""
    d, nlist, pq_m = args.d, args.nlist, args.pq_m
    dsub = d // pq_m
    if args.dtype == "u8":
        c = synth.sift_like_centroids(nlist, d)
        scale = 20.0
    else:
        c = synth.deep_like_centroids(nlist, d)
        scale = 0.05
    ct = torch.from_numpy(c).cuda()
    cb = torch.from_numpy(synth.pq_codebooks(pq_m, dsub, scale, seed=1)).cuda()
    rows = []
    done = 0
    chunk = 0
    while done < args.n:
        take = min(synth.CHUNK_ROWS, args.n - done)
        x = synth.sift_like_rows(chunk, rows=take, d=d) if args.dtype == "u8" else synth.deep_like_rows(chunk, take, d)
        rows.append(torch.from_numpy(x).cuda())
        done += take
        chunk += 1
    xt = torch.cat(rows)
    del rows
    ids, _ = B.ivf_assign(xt, ct)
    xr, offsets, order = B.ivf_cluster_major_reorder(xt, ids, nlist)
    ids_sorted = ids[order.long()]
    del xt
    B.ivf_pq_encode(xr[:1024], ids_sorted[:1024], ct, cb)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    codes = B.ivf_pq_encode(xr, ids_sorted, ct, cb)
    e1.record()
    B.ivf_check()
    enc_ms = e0.elapsed_time(e1)
    lens = (offsets[1:] - offsets[:-1]).float()
    out = {"op": "pq", "n": args.n, "nlist": nlist, "d": d, "pq_m": pq_m, "dtype": args.dtype, "nprobe": args.k,
           "n_rerank": args.n_rerank, "encode_ms": enc_ms, "encode_vectors_per_s": args.n / (enc_ms / 1e3),
           "list_len": {"mean": lens.mean().item(), "max": lens.max().item(), "empty": int((lens == 0).sum().item())},
           "batches": {}}
    bmax = max(int(v) for v in args.batches.split(","))
    q_all = synth.sift_like_queries(bmax, d) if args.dtype == "u8" else synth.deep_like_queries(bmax, d)
    handle = B.PreparedCentroids(ct)
    for bs in [int(v) for v in args.batches.split(",")]:
        q = torch.from_numpy(q_all[:bs]).cuda()
        probes = torch.empty((bs, args.k), dtype=torch.int32, device="cuda")
        B.ivf_route_prepared(handle, q, args.k, probes, None, want_dists=False)
        for _ in range(3):
            pos, est, cnt = B.ivf_pq_search(q, ct, probes, offsets, codes, cb, args.n_rerank)
        B.ivf_check()
        reps = max(args.reps, 10)
        B.ivf_debug_timing(True)
        e0.record()
        for _ in range(reps):
            B.ivf_pq_search(q, ct, probes, offsets, codes, cb, args.n_rerank)
        e1.record()
        fam = B.ivf_debug_timing_read()
        B.ivf_debug_timing(False)
        us = e0.elapsed_time(e1) / reps * 1e3
        e0.record()
        for _ in range(reps):
            B.ivf_route_prepared(handle, q, args.k, probes, None, want_dists=False)
            B.ivf_pq_search(q, ct, probes, offsets, codes, cb, args.n_rerank)
        e1.record()
        B.ivf_check()
        both_us = e0.elapsed_time(e1) / reps * 1e3
        scanned = int(cnt.sum().item())
        out["batches"][str(bs)] = {
            "search_us": us, "route_plus_search_us": both_us, "queries_per_s": bs / (both_us / 1e6),
            "codes_scanned": scanned, "codes_per_s": scanned / (us / 1e6),
            "lookups_per_s": scanned * pq_m / (us / 1e6), "code_GBps": scanned * pq_m / (us / 1e6) / 1e9,
            "kernel_us": {k: v[0] / max(v[1], 1) * 1e3 for k, v in fam.items() if v[1]}}
    handle.close()
    print(json.dumps(out))


def candidates_case(args):
    """Assignment within --k given candidates per row (random candidates: the gather is what costs)."""
    x = synth.sift_like_rows(0, rows=args.n, d=args.d) if args.dtype == "u8" else synth.deep_like_rows(0, args.n, args.d)
    c = synth.sift_like_centroids(args.nlist, args.d) if args.dtype == "u8" else synth.deep_like_centroids(args.nlist, args.d)
    xt, ct = torch.from_numpy(x).cuda(), torch.from_numpy(c).cuda()
    cand = torch.randint(0, args.nlist, (args.n, args.k), dtype=torch.int32, device="cuda",
                         generator=torch.Generator(device="cuda").manual_seed(1))
    for _ in range(3):
        B.ivf_assign_candidates(xt, ct, cand)
    B.ivf_check()
    reps = max(args.reps, 10)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        B.ivf_assign_candidates(xt, ct, cand)
    e1.record()
    B.ivf_check()
    ms = e0.elapsed_time(e1) / reps
    esize = 1 if args.dtype == "u8" else 4
    nbytes = args.n * (args.d * esize + args.k * 4 + args.k * args.d * 4 + 8)
    print(json.dumps({"op": "candidates", "n": args.n, "nlist": args.nlist, "d": args.d, "m": args.k, "dtype": args.dtype,
                      "ms_per_call": ms, "vectors_per_s": args.n / (ms / 1e3), "algorithmic_GBps": nbytes / (ms / 1e3) / 1e9}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="assign", choices=["assign", "route", "update", "stream", "serve", "pq", "candidates", "build"])
    ap.add_argument("--train-rows", type=int, default=1 << 20, dest="train_rows", help="sample size of --op build")
    ap.add_argument("--pq-m", type=int, default=32, dest="pq_m")
    ap.add_argument("--n-rerank", type=int, default=512, dest="n_rerank")
    ap.add_argument("--batches", default="8,32,256,2048", help="query batch sizes of --op serve")
    ap.add_argument("--iters", type=int, default=1, help="Lloyd iterations of --op stream")
    ap.add_argument("--check-rows", type=int, default=0, dest="check_rows",
                    help="--op stream: seeded rows per iteration handed to the checker callback, if one is given")
    ap.add_argument("--n", type=int, default=262144)
    ap.add_argument("--nlist", type=int, default=65536)
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--k", type=int, default=64)
    ap.add_argument("--dtype", default="u8", choices=["u8", "f32", "i8"])
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--dependent-launch", type=int, default=-1, help="kernel-family mask of dependent launches (0 = none)")
    ap.add_argument("--crossing-cost", type=int, default=-1, help="span-partition crossing cost in units (0 = equal counts)")
    ap.add_argument("--rotation", type=int, default=1, help="0 = centroid tiles swept in index order (for comparison)")
    ap.add_argument("--split-threshold-pass", type=int, default=0, dest="split_threshold",
                    help="1 = threshold pass always as sketch kernel + merge launch (for comparison)")
    args = ap.parse_args()
    B.ivf_debug_set_rotation(bool(args.rotation))
    B.ivf_debug_set_threshold_pass(bool(args.split_threshold))
    if args.crossing_cost >= 0:
        B.ivf_debug_set_crossing_cost(args.crossing_cost)
    if args.dependent_launch >= 0:
        B.ivf_debug_set_dependent_launch(args.dependent_launch)

    if args.op == "stream":
        return stream_case(args)
    if args.op == "serve":
        return serve_case(args)
    if args.op == "pq":
        return pq_case(args)
    if args.op == "candidates":
        return candidates_case(args)
    if args.op == "build":
        return build_case(args)
    if args.dtype == "i8":
        x, c = synth.spacev_like(args.n, args.nlist, seed=0, d=args.d)
    elif args.dtype == "u8":
        x = synth.sift_like_rows(0, rows=args.n, d=args.d)
        c = synth.sift_like_centroids(args.nlist, args.d)
    else:
        x = synth.deep_like_rows(0, rows=args.n, d=args.d)
        c = synth.deep_like_centroids(args.nlist, args.d)
    xt, ct = torch.from_numpy(x).cuda(), torch.from_numpy(c).cuda()
    k = 1 if args.op != "route" else args.k
    ids = torch.empty((args.n, k) if k > 1 else (args.n,), dtype=torch.int32, device="cuda")
    dists = torch.empty_like(ids, dtype=torch.float32)
    sums = torch.zeros((args.nlist, args.d), dtype=torch.float32, device="cuda")
    counts = torch.zeros((args.nlist,), dtype=torch.int64, device="cuda")
    if args.op == "update":
        ids = torch.from_numpy(np.random.default_rng(0).integers(0, args.nlist, args.n).astype(np.int32)).cuda()

    def call():
        if args.op == "assign":
            B.ivf_assign(xt, ct, ids, dists)
        elif args.op == "route":
            B.ivf_route(xt, ct, k, ids, dists)
        else:
            B.ivf_centroid_update(xt, ids, sums, counts)

    call()
    B.ivf_check()
    B.ivf_debug_stats(True)
    call()
    stats = B.ivf_debug_stats(False)
    B.ivf_debug_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        call()
    e1.record()
    fam = B.ivf_debug_timing_read()
    B.ivf_check()
    flops = 2.0 * args.n * args.nlist * args.d
    out = {"op": args.op, "n": args.n, "nlist": args.nlist, "d": args.d, "k": k, "dtype": args.dtype,
           "ms_per_call": e0.elapsed_time(e1) / args.reps,
           "kernel_ms": {name: ms / max(cnt, 1) for name, (ms, cnt) in fam.items() if cnt}}
    fused = out["kernel_ms"].get("fused_argmin") or out["kernel_ms"].get("fused_topk")
    if k > 1:
        out["stats_per_call"] = stats
    if fused:
        out["fused_tflops"] = flops / (fused / 1e3) / 1e12
    print(json.dumps(out))


if __name__ == "__main__":
    main()
