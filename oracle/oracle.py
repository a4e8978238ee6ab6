"""ctypes face of the CPU oracle (``ivf_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg load
this; the product path never does.  The arithmetic is all in the C file; this module only
marshals numpy arrays and compiles the C on first use (gcc, -O2, OpenMP over rows).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ivf_oracle.c")
_SRC_PQ = os.path.join(_HERE, "pq_oracle.c")
_LIB = os.path.join(_HERE, "libivf_oracle.so")

F32, U8, I8 = 0, 1, 2
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object next to it."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_PQ))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", _SRC, _SRC_PQ, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, i32, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
        _lib.oracle_route.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, i32, i32, vp, vp, vp]
        _lib.oracle_assign.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, i32, vp, vp]
        _lib.oracle_pair_dists.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, i64, vp, vp, vp]
        _lib.oracle_sqnorms.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp]
        _lib.oracle_update.argtypes = [vp, ctypes.c_int, vp, i64, ctypes.c_int, i32, vp, vp]
        _lib.oracle_finalize.argtypes = [vp, vp, i32, ctypes.c_int, vp]
        _lib.oracle_reorder.argtypes = [vp, i64, i32, vp, vp]
        _lib.oracle_lloyd.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, i32, ctypes.c_int, vp, vp, vp]
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_assign_candidates.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, i32, vp, ctypes.c_int, vp, vp]
        _lib.oracle_pq_lut.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, vp]
        _lib.oracle_pq_lut.restype = None
        _lib.oracle_pq_adc.argtypes = [vp, ctypes.c_int, vp, i64, i64, vp]
        _lib.oracle_pq_adc.restype = None
        _lib.oracle_residuals.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, vp, i32, vp]
        _lib.oracle_pq_encode.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, vp, i32, vp, ctypes.c_int, vp]
        _lib.oracle_pq_search.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp, i32, vp, ctypes.c_int, vp, vp,
                                          vp, ctypes.c_int, ctypes.c_int, vp, vp, vp]
    return _lib


def _rows(x: np.ndarray):
    """(contiguous array, dtype code) for a float32, uint8 or int8 row matrix."""
    if x.dtype == np.uint8:
        return np.ascontiguousarray(x), U8
    if x.dtype == np.int8:
        return np.ascontiguousarray(x), I8
    if x.dtype == np.float32:
        return np.ascontiguousarray(x), F32
    raise TypeError(f"oracle takes float32, uint8 or int8 rows, got {x.dtype}")


def _cent(c: np.ndarray) -> np.ndarray:
    if c.dtype != np.float32:
        raise TypeError("centroids must be float32")
    return np.ascontiguousarray(c)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def route(x: np.ndarray, c: np.ndarray, k: int):
    """(ids [n,k] int32, dists [n,k] float64, next [n] float64): the k nearest centroids of every
    row in ascending (distance, id) order and the (k+1)-th distance."""
    x, xt = _rows(x)
    c = _cent(c)
    n, d = x.shape
    nlist = c.shape[0]
    assert c.shape[1] == d
    ids = np.empty((n, k), np.int32)
    dists = np.empty((n, k), np.float64)
    nxt = np.empty((n,), np.float64)
    rc = _load().oracle_route(_p(x), xt, n, d, _p(c), nlist, k, _p(ids), _p(dists), _p(nxt))
    if rc != 0:
        raise ValueError("oracle_route: bad arguments")
    return ids, dists, nxt


def assign(x: np.ndarray, c: np.ndarray):
    """(ids [n] int32, dists [n] float64): nearest centroid of every row."""
    x, xt = _rows(x)
    c = _cent(c)
    n, d = x.shape
    ids = np.empty((n,), np.int32)
    dists = np.empty((n,), np.float64)
    rc = _load().oracle_assign(_p(x), xt, n, d, _p(c), c.shape[0], _p(ids), _p(dists))
    if rc != 0:
        raise ValueError("oracle_assign: bad arguments")
    return ids, dists


def assign_candidates(x: np.ndarray, c: np.ndarray, cand: np.ndarray):
    """(ids [n] int32, dists [n] float64): the nearest centroid among each row's candidates cand [n, m]."""
    x, xt = _rows(x)
    c = _cent(c)
    cand = np.ascontiguousarray(cand, np.int32)
    n, d = x.shape
    assert cand.shape[0] == n
    ids = np.empty((n,), np.int32)
    dists = np.empty((n,), np.float64)
    rc = _load().oracle_assign_candidates(_p(x), xt, n, d, _p(c), c.shape[0], _p(cand), cand.shape[1], _p(ids), _p(dists))
    if rc != 0:
        raise ValueError("oracle_assign_candidates: bad arguments")
    return ids, dists


def pair_dists(x: np.ndarray, c: np.ndarray, rows: np.ndarray, cols: np.ndarray) -> np.ndarray:
    """Squared distances of the given (row of x, row of c) pairs, float64."""
    x, xt = _rows(x)
    c = _cent(c)
    rows = np.ascontiguousarray(rows, np.int64)
    cols = np.ascontiguousarray(cols, np.int32)
    out = np.empty(rows.shape, np.float64)
    _load().oracle_pair_dists(_p(x), xt, x.shape[1], _p(c), rows.size, _p(rows), _p(cols), _p(out))
    return out


def sqnorms(x: np.ndarray) -> np.ndarray:
    x, xt = _rows(x)
    out = np.empty((x.shape[0],), np.float64)
    _load().oracle_sqnorms(_p(x), xt, x.shape[0], x.shape[1], _p(out))
    return out


def update(x: np.ndarray, ids: np.ndarray, nlist: int, sums: np.ndarray | None = None,
           counts: np.ndarray | None = None):
    """Accumulate per-list sums (float64 [nlist,d]) and counts (int64 [nlist]); returns
    (sums, counts, ok) where ok is False if some id was out of range (that row is skipped)."""
    x, xt = _rows(x)
    n, d = x.shape
    ids = np.ascontiguousarray(ids, np.int32)
    if sums is None:
        sums = np.zeros((nlist, d), np.float64)
    if counts is None:
        counts = np.zeros((nlist,), np.int64)
    assert sums.dtype == np.float64 and counts.dtype == np.int64 and sums.flags.c_contiguous
    rc = _load().oracle_update(_p(x), xt, _p(ids), n, d, nlist, _p(sums), _p(counts))
    return sums, counts, rc == 0


def reorder(ids: np.ndarray, nlist: int):
    """(offsets int64 [nlist+1], order int64 [n]): cluster-major layout, input order kept inside a list."""
    ids = np.ascontiguousarray(ids, np.int32)
    offsets = np.empty((nlist + 1,), np.int64)
    order = np.empty((ids.shape[0],), np.int64)
    rc = _load().oracle_reorder(_p(ids), ids.shape[0], nlist, _p(offsets), _p(order))
    if rc != 0:
        raise ValueError("oracle_reorder: id out of range")
    return offsets, order


def finalize(sums: np.ndarray, counts: np.ndarray, centroids: np.ndarray) -> np.ndarray:
    """New float32 centroids: mean per list, empty lists keep the row of ``centroids``."""
    out = np.array(centroids, dtype=np.float32, order="C", copy=True)
    sums = np.ascontiguousarray(sums, np.float64)
    counts = np.ascontiguousarray(counts, np.int64)
    _load().oracle_finalize(_p(sums), _p(counts), out.shape[0], out.shape[1], _p(out))
    return out


def lloyd(x: np.ndarray, init_centroids: np.ndarray, iters: int):
    """(centroids float32, ids int32 of the last iteration, inertia float64 [iters])."""
    x, xt = _rows(x)
    c = np.array(init_centroids, dtype=np.float32, order="C", copy=True)
    n, d = x.shape
    ids = np.empty((n,), np.int32)
    inertia = np.empty((iters,), np.float64)
    rc = _load().oracle_lloyd(_p(x), xt, n, d, c.shape[0], iters, _p(c), _p(ids), _p(inertia))
    if rc != 0:
        raise ValueError("oracle_lloyd failed")
    return c, ids, inertia


# ---------------------------------------------------------------- residual-PQ candidate reduction
def _codebooks(cb: np.ndarray, d: int):
    """codebooks [pq_m, 256, d // pq_m] float32"""
    if cb.dtype != np.float32 or cb.ndim != 3 or cb.shape[1] != 256 or cb.shape[0] * cb.shape[2] != d:
        raise TypeError("codebooks must be float32 [pq_m, 256, d / pq_m]")
    return np.ascontiguousarray(cb), cb.shape[0]


def pq_lut(r: np.ndarray, codebooks: np.ndarray) -> np.ndarray:
    """float32 [pq_m, 256] table of one residual r [d] (float32)."""
    r = np.ascontiguousarray(r, np.float32)
    cb, m = _codebooks(codebooks, r.shape[0])
    lut = np.empty((m, 256), np.float32)
    _load().oracle_pq_lut(_p(r), r.shape[0], m, _p(cb), _p(lut))
    return lut


def pq_adc(lut: np.ndarray, codes: np.ndarray) -> np.ndarray:
    """float32 ADC estimates of codes [n, pq_m] (uint8) with one table."""
    lut = np.ascontiguousarray(lut, np.float32)
    codes = np.ascontiguousarray(codes, np.uint8)
    est = np.empty((codes.shape[0],), np.float32)
    _load().oracle_pq_adc(_p(lut), lut.shape[0], _p(codes), 0, codes.shape[0], _p(est))
    return est


def pq_encode(x: np.ndarray, ids: np.ndarray, c: np.ndarray, codebooks: np.ndarray) -> np.ndarray:
    """uint8 [n, pq_m]: residual-PQ codes of the rows of x, row i assigned to list ids[i]."""
    x, xt = _rows(x)
    c = _cent(c)
    n, d = x.shape
    cb, m = _codebooks(codebooks, d)
    ids = np.ascontiguousarray(ids, np.int32)
    codes = np.empty((n, m), np.uint8)
    rc = _load().oracle_pq_encode(_p(x), xt, n, d, _p(ids), _p(c), c.shape[0], _p(cb), m, _p(codes))
    if rc != 0:
        raise ValueError("oracle_pq_encode: bad arguments")
    return codes


def pq_search(q: np.ndarray, c: np.ndarray, probes: np.ndarray, offsets: np.ndarray, codes: np.ndarray,
              codebooks: np.ndarray, n_rerank: int):
    """(pos int64 [nq, n_rerank], est float32 [nq, n_rerank], count int64 [nq]): the n_rerank smallest
    ADC estimates over the codes of every query's probed lists, ascending (estimate, position)."""
    q, qt = _rows(q)
    c = _cent(c)
    nq, d = q.shape
    cb, m = _codebooks(codebooks, d)
    probes = np.ascontiguousarray(probes, np.int32)
    offsets = np.ascontiguousarray(offsets, np.int64)
    codes = np.ascontiguousarray(codes, np.uint8)
    assert probes.shape[0] == nq and offsets.shape[0] == c.shape[0] + 1 and codes.shape[1] == m
    pos = np.empty((nq, n_rerank), np.int64)
    est = np.empty((nq, n_rerank), np.float32)
    count = np.empty((nq,), np.int64)
    rc = _load().oracle_pq_search(_p(q), qt, nq, d, _p(c), c.shape[0], _p(probes), probes.shape[1], _p(offsets),
                                  _p(codes), _p(cb), m, n_rerank, _p(pos), _p(est), _p(count))
    if rc != 0:
        raise ValueError("oracle_pq_search: bad arguments")
    return pos, est, count


def residuals(x: np.ndarray, ids: np.ndarray, c: np.ndarray) -> np.ndarray:
    """float32 [n, d]: x - c[ids], one rounded fp32 subtraction per coordinate."""
    x, xt = _rows(x)
    c = _cent(c)
    ids = np.ascontiguousarray(ids, np.int32)
    out = np.empty(x.shape, np.float32)
    rc = _load().oracle_residuals(_p(x), xt, x.shape[0], x.shape[1], _p(ids), _p(c), c.shape[0], _p(out))
    if rc != 0:
        raise ValueError("oracle_residuals: id out of range")
    return out
