"""Python face of the C-ABI library (``include/ivf_b200.h``): argument marshalling only.

Every function takes torch tensors (CUDA tensors, or page-locked CPU tensors where the C function
accepts host memory), checks dtype / shape / contiguity, and passes raw pointers and sizes plus
the current CUDA stream to the library.  No step of the computation runs in Python or in torch.
There is no fallback: if the library cannot be loaded the import of a symbol raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

IVF_F32, IVF_U8, IVF_I8 = 0, 1, 2
IVF_OK = 0
IVF_ERR_INVALID_ARG, IVF_ERR_UNSUPPORTED, IVF_ERR_ALLOC = -1, -2, -3
IVF_ERR_CUDA, IVF_ERR_DEVICE_TIMEOUT, IVF_ERR_BAD_ID, IVF_ERR_BOUNDS = -4, -5, -6, -7

EXPORTS = (
    "ivf_route", "ivf_assign", "ivf_centroid_update", "ivf_centroid_update_noalloc", "ivf_centroid_finalize",
    "ivf_assign_update", "ivf_cluster_major_reorder", "ivf_centroids_create", "ivf_centroids_destroy",
    "ivf_route_prepared",
    "ivf_pq_encode", "ivf_pq_search", "ivf_pq_residuals", "ivf_assign_candidates", "ivf_merge_shards",
    "ivf_set_deferred_host_outputs", "ivf_wait_host_outputs",
    "ivf_check", "ivf_last_error", "ivf_release_workspace", "ivf_launch_count",
    "ivf_debug_plan", "ivf_debug_span", "ivf_debug_rotation", "ivf_debug_set_rotation", "ivf_debug_set_threshold_pass", "ivf_debug_fail_next_alloc", "ivf_debug_bounds_checked", "ivf_debug_bounds_probe", "ivf_debug_set_wait_limit_ns",
    "ivf_debug_timing", "ivf_debug_timing_read", "ivf_debug_wait_probe", "ivf_debug_force_fallback", "ivf_debug_rule", "ivf_debug_set_row_chunk", "ivf_debug_stats", "ivf_debug_set_pq_groups", "ivf_debug_set_dependent_launch", "ivf_debug_set_crossing_cost",
)

_lib = None


class IvfError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"ivf_b200 error {code}: {message}")
        self.code = code


def lib() -> ctypes.CDLL:
    """The loaded shared library; built in-tree first if it is missing or older than its sources."""
    global _lib
    if _lib is not None:
        return _lib
    # IVF_B200_CHECKED=1 selects the build whose kernels check their indices (see ivf_debug_bounds_checked)
    checked = os.environ.get("IVF_B200_CHECKED", "0") not in ("", "0")
    path = _build.CHECKED_LIB_PATH if checked else _build.LIB_PATH
    if not os.path.exists(path) or _build._stale(path):
        try:
            path = _build.build(checked=checked)
        except Exception as exc:  # no nvcc on this machine: use what travelled with the tree
            if not os.path.exists(path):
                raise RuntimeError(f"libivf_b200.so is missing and could not be built: {exc}") from exc
    L = ctypes.CDLL(path)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    L.ivf_route.argtypes = [vp, i64, i32, i32, vp, i32, i32, vp, vp, vp]
    L.ivf_assign.argtypes = [vp, i64, i32, i32, vp, i32, vp, vp, vp]
    L.ivf_set_deferred_host_outputs.argtypes = [i32]
    L.ivf_wait_host_outputs.argtypes = [vp]
    L.ivf_centroid_update.argtypes = [vp, i32, vp, i64, i32, i32, vp, vp, vp]
    L.ivf_centroid_update_noalloc.argtypes = [vp, i32, vp, i64, i32, i32, vp, vp, vp]
    L.ivf_centroid_finalize.argtypes = [vp, vp, i32, i32, vp, vp]
    L.ivf_cluster_major_reorder.argtypes = [vp, i32, vp, i64, i32, i32, vp, vp, vp, vp]
    L.ivf_centroids_create.argtypes = [vp, i32, i32, ctypes.POINTER(vp), vp]
    L.ivf_centroids_destroy.argtypes = [vp, vp]
    L.ivf_route_prepared.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp]
    L.ivf_assign_update.argtypes = [vp, i64, i32, i32, vp, i32, vp, vp, vp, vp, i64, vp]
    L.ivf_check.argtypes = [vp]
    L.ivf_last_error.restype = ctypes.c_char_p
    L.ivf_launch_count.restype = i64
    L.ivf_debug_plan.argtypes = [i64, i32, i32, i32, i32, ctypes.POINTER(i64)]
    L.ivf_debug_span.argtypes = [i64, i32, i32, i32, i32, i32, ctypes.POINTER(i64)]
    L.ivf_debug_rotation.argtypes = [i64, i32, i32, i32, i32, i64]
    L.ivf_debug_set_wait_limit_ns.argtypes = [i64]
    L.ivf_debug_fail_next_alloc.argtypes = [i32]
    L.ivf_debug_bounds_probe.argtypes = [vp]
    L.ivf_debug_timing.argtypes = [i32]
    L.ivf_debug_wait_probe.argtypes = [vp]
    L.ivf_debug_force_fallback.argtypes = [i32]
    L.ivf_debug_set_row_chunk.argtypes = [i64]
    L.ivf_debug_stats.argtypes = [i32, ctypes.POINTER(i64)]
    L.ivf_debug_rule.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_int)]
    L.ivf_assign_candidates.argtypes = [vp, i64, i32, i32, vp, i32, vp, i32, vp, vp, vp]
    L.ivf_merge_shards.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
    L.ivf_pq_residuals.argtypes = [vp, i64, i32, i32, vp, vp, i32, vp, vp]
    L.ivf_pq_encode.argtypes = [vp, i64, i32, i32, vp, vp, i32, vp, i32, vp, vp]
    L.ivf_pq_search.argtypes = [vp, i64, i32, i32, vp, i32, vp, i32, vp, vp, i64, vp, i32, i32, vp, vp, vp, vp, vp]
    L.ivf_debug_set_pq_groups.argtypes = [i32]
    L.ivf_debug_set_crossing_cost.argtypes = [i32]
    L.ivf_debug_set_dependent_launch.argtypes = [i32]
    L.ivf_debug_timing_read.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    for name in EXPORTS:
        if name not in ("ivf_last_error", "ivf_launch_count"):
            getattr(L, name).restype = i32
    _lib = L
    return L


def _raise(code: int):
    raise IvfError(code, lib().ivf_last_error().decode())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return IVF_F32
    if t.dtype == torch.uint8:
        return IVF_U8
    if t.dtype == torch.int8:
        return IVF_I8
    raise TypeError(f"points must be float32, uint8 or int8, got {t.dtype}")


def _rows(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.dim() != 2 or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous 2-D tensor")
    if not (t.is_cuda or t.is_pinned()):
        raise ValueError(f"{name} must be a CUDA tensor or a pinned CPU tensor")
    return t


def _dev(t: torch.Tensor, name: str, dtype: torch.dtype) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    return t


def _out(t: torch.Tensor, name: str, dtype: torch.dtype) -> torch.Tensor:
    """An output array: a contiguous CUDA tensor, or a pinned CPU tensor (results read back by the library)."""
    if not (t.is_cuda or t.is_pinned()) or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA or pinned CPU tensor of {dtype}")
    return t


def _stream(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def ivf_route(queries: torch.Tensor, centroids: torch.Tensor, nprobe: int,
              out_ids: torch.Tensor | None = None, out_dists: torch.Tensor | None = None,
              want_dists: bool = True):
    """ids [nq, nprobe] int32 (and squared distances [nq, nprobe] float32) of the nprobe nearest
    centroids of every query, ascending by (distance, id).  Enqueued on the current stream."""
    _rows(queries, "queries")
    _dev(centroids, "centroids", torch.float32)
    nq, d = queries.shape
    nlist = centroids.shape[0]
    dev = centroids.device
    if out_ids is None:
        out_ids = torch.empty((nq, nprobe), dtype=torch.int32, device=dev)
    if out_dists is None and want_dists:
        out_dists = torch.empty((nq, nprobe), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_route(_ptr(queries), nq, d, _dtype_code(queries), _ptr(centroids), nlist, nprobe,
                             _ptr(_out(out_ids, "out_ids", torch.int32)),
                             _ptr(None if out_dists is None else _out(out_dists, "out_dists", torch.float32)), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_dists


class PreparedCentroids:
    """Handle of a device-resident prepared centroid table (ivf_centroids_create / _destroy)."""

    def __init__(self, centroids: torch.Tensor):
        _dev(centroids, "centroids", torch.float32)
        self.nlist, self.d = centroids.shape
        self.device = centroids.device
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib().ivf_centroids_create(_ptr(centroids), self.nlist, self.d, ctypes.byref(self._h),
                                            _stream(self.device))
        if rc != IVF_OK:
            _raise(rc)

    def close(self):
        if self._h:
            with torch.cuda.device(self.device):
                lib().ivf_centroids_destroy(self._h, _stream(self.device))
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ivf_route_prepared(handle: PreparedCentroids, queries: torch.Tensor, nprobe: int,
                       out_ids: torch.Tensor | None = None, out_dists: torch.Tensor | None = None,
                       want_dists: bool = True):
    """ivf_route against a prepared, device-resident centroid table."""
    _rows(queries, "queries")
    nq, d = queries.shape
    if d != handle.d:
        raise ValueError("dimension mismatch between queries and the prepared centroids")
    dev = handle.device
    if out_ids is None:
        out_ids = torch.empty((nq, nprobe), dtype=torch.int32, device=dev)
    if out_dists is None and want_dists:
        out_dists = torch.empty((nq, nprobe), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_route_prepared(handle._h, _ptr(queries), nq, _dtype_code(queries), nprobe,
                                      _ptr(_out(out_ids, "out_ids", torch.int32)),
                                      _ptr(None if out_dists is None else _out(out_dists, "out_dists", torch.float32)),
                                      _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_dists


def ivf_assign(points: torch.Tensor, centroids: torch.Tensor,
               out_ids: torch.Tensor | None = None, out_dists: torch.Tensor | None = None,
               want_dists: bool = True):
    """ids [n] int32 (and squared distances [n] float32) of the nearest centroid of every row."""
    _rows(points, "points")
    _dev(centroids, "centroids", torch.float32)
    n, d = points.shape
    dev = centroids.device
    if out_ids is None:
        out_ids = torch.empty((n,), dtype=torch.int32, device=dev)
    if out_dists is None and want_dists:
        out_dists = torch.empty((n,), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_assign(_ptr(points), n, d, _dtype_code(points), _ptr(centroids), centroids.shape[0],
                              _ptr(_out(out_ids, "out_ids", torch.int32)),
                              _ptr(None if out_dists is None else _out(out_dists, "out_dists", torch.float32)), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_dists


def ivf_set_deferred_host_outputs(on: bool, device=None) -> None:
    """Calls with pinned-host outputs stop making the stream wait for their read-back (per device)."""
    with torch.cuda.device(device if device is not None else torch.cuda.current_device()):
        rc = lib().ivf_set_deferred_host_outputs(1 if on else 0)
    if rc != IVF_OK:
        _raise(rc)


def ivf_wait_host_outputs(device=None) -> None:
    """Makes the current stream wait for every read-back issued so far on the device."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        rc = lib().ivf_wait_host_outputs(_stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_centroid_update(points: torch.Tensor, ids: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor):
    """sums[l] += member rows, counts[l] += members; accumulates in place (all CUDA tensors)."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(ids, "ids", torch.int32)
    _dev(sums, "sums", torch.float32)
    _dev(counts, "counts", torch.int64)
    n, d = points.shape
    nlist = sums.shape[0]
    if sums.shape != (nlist, d) or counts.shape != (nlist,) or ids.shape != (n,):
        raise ValueError("shape mismatch between points, ids, sums and counts")
    dev = points.device
    with torch.cuda.device(dev):
        rc = lib().ivf_centroid_update(_ptr(points), _dtype_code(points), _ptr(ids), n, d, nlist,
                                       _ptr(sums), _ptr(counts), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_centroid_update_noalloc(points: torch.Tensor, ids: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor):
    """ivf_centroid_update for callers that must not allocate device memory at call time (for
    instance beside a serving process whose pool already owns all free memory): the library's
    built-in scratch is used, so at most 1,048,576 rows and 65,536 lists per call.  Calls on one
    device share that scratch and must not overlap on the GPU."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(ids, "ids", torch.int32)
    _dev(sums, "sums", torch.float32)
    _dev(counts, "counts", torch.int64)
    n, d = points.shape
    nlist = sums.shape[0]
    if sums.shape != (nlist, d) or counts.shape != (nlist,) or ids.shape != (n,):
        raise ValueError("shape mismatch between points, ids, sums and counts")
    dev = points.device
    with torch.cuda.device(dev):
        rc = lib().ivf_centroid_update_noalloc(_ptr(points), _dtype_code(points), _ptr(ids), n, d, nlist,
                                               _ptr(sums), _ptr(counts), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_cluster_major_reorder(points: torch.Tensor, ids: torch.Tensor, nlist: int):
    """(out_points [n,d], out_offsets int64 [nlist+1], out_order int32 [n]): the rows regrouped so that
    every list is contiguous; the order inside a list is unspecified."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(ids, "ids", torch.int32)
    n, d = points.shape
    dev = points.device
    out_points = torch.empty_like(points)
    out_offsets = torch.empty((nlist + 1,), dtype=torch.int64, device=dev)
    out_order = torch.empty((n,), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_cluster_major_reorder(_ptr(points), _dtype_code(points), _ptr(ids), n, d, nlist,
                                             _ptr(out_points), _ptr(out_offsets), _ptr(out_order), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_points, out_offsets, out_order


def ivf_assign_candidates(points: torch.Tensor, centroids: torch.Tensor, cand_ids: torch.Tensor,
                          want_dists: bool = True):
    """(ids int32 [n], dists float32 [n] or None): for every row the nearest centroid among its
    candidates cand_ids [n, m] (exact squared L2 within the set)."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(centroids, "centroids", torch.float32)
    _dev(cand_ids, "cand_ids", torch.int32)
    n, d = points.shape
    if cand_ids.dim() != 2 or cand_ids.shape[0] != n:
        raise ValueError("cand_ids must be [n, m]")
    dev = points.device
    out_ids = torch.empty((n,), dtype=torch.int32, device=dev)
    out_dists = torch.empty((n,), dtype=torch.float32, device=dev) if want_dists else None
    with torch.cuda.device(dev):
        rc = lib().ivf_assign_candidates(_ptr(points), n, d, _dtype_code(points), _ptr(centroids), centroids.shape[0],
                                         _ptr(cand_ids), cand_ids.shape[1], _ptr(out_ids), _ptr(out_dists), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_dists


def ivf_merge_shards(shard_ids: torch.Tensor, shard_dists: torch.Tensor):
    """[parts, nq, k] per-shard routing results (global ids) -> (ids [nq, k] int32, dists [nq, k] float32):
    the k smallest pairs by (distance, id) per query."""
    _dev(shard_ids, "shard_ids", torch.int32)
    _dev(shard_dists, "shard_dists", torch.float32)
    if shard_ids.dim() != 3 or shard_ids.shape != shard_dists.shape:
        raise ValueError("shard_ids and shard_dists must both be [parts, nq, k]")
    parts, nq, k = shard_ids.shape
    dev = shard_ids.device
    out_ids = torch.empty((nq, k), dtype=torch.int32, device=dev)
    out_dists = torch.empty((nq, k), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_merge_shards(_ptr(shard_ids), _ptr(shard_dists), parts, nq, k, _ptr(out_ids), _ptr(out_dists),
                                    _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_dists


def _codebooks(codebooks: torch.Tensor, d: int) -> int:
    _dev(codebooks, "codebooks", torch.float32)
    if codebooks.dim() != 3 or codebooks.shape[1] != 256 or codebooks.shape[0] * codebooks.shape[2] != d:
        raise ValueError("codebooks must be [pq_m, 256, d / pq_m]")
    return codebooks.shape[0]


def ivf_pq_residuals(points: torch.Tensor, ids: torch.Tensor, centroids: torch.Tensor) -> torch.Tensor:
    """float32 [n, d]: points - centroids[ids], the training vectors of the PQ codebooks."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(ids, "ids", torch.int32)
    _dev(centroids, "centroids", torch.float32)
    n, d = points.shape
    out = torch.empty((n, d), dtype=torch.float32, device=points.device)
    with torch.cuda.device(points.device):
        rc = lib().ivf_pq_residuals(_ptr(points), n, d, _dtype_code(points), _ptr(ids), _ptr(centroids),
                                    centroids.shape[0], _ptr(out), _stream(points.device))
    if rc != IVF_OK:
        _raise(rc)
    return out


def ivf_pq_encode(points: torch.Tensor, ids: torch.Tensor, centroids: torch.Tensor, codebooks: torch.Tensor):
    """uint8 [n, pq_m] residual-PQ codes of the rows of points, row i assigned to list ids[i]."""
    if not points.is_cuda:
        raise ValueError("points must be a CUDA tensor")
    _rows(points, "points")
    _dev(ids, "ids", torch.int32)
    _dev(centroids, "centroids", torch.float32)
    n, d = points.shape
    pq_m = _codebooks(codebooks, d)
    dev = points.device
    codes = torch.empty((n, pq_m), dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ivf_pq_encode(_ptr(points), n, d, _dtype_code(points), _ptr(ids), _ptr(centroids),
                                 centroids.shape[0], _ptr(codebooks), pq_m, _ptr(codes), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return codes


def ivf_pq_search(queries: torch.Tensor, centroids: torch.Tensor, probe_ids: torch.Tensor, list_offsets: torch.Tensor,
                  codes: torch.Tensor, codebooks: torch.Tensor, n_rerank: int, vec_ids: torch.Tensor | None = None,
                  want_counts: bool = True):
    """(ids int64 [nq, n_rerank], estimates float32 [nq, n_rerank], counts int64 [nq] or None): the
    n_rerank smallest ADC estimates over the codes of every query's probed lists, ascending."""
    if not queries.is_cuda:
        raise ValueError("queries must be a CUDA tensor")
    _rows(queries, "queries")
    _dev(centroids, "centroids", torch.float32)
    _dev(probe_ids, "probe_ids", torch.int32)
    _dev(list_offsets, "list_offsets", torch.int64)
    _dev(codes, "codes", torch.uint8)
    if vec_ids is not None:
        _dev(vec_ids, "vec_ids", torch.int64)
    nq, d = queries.shape
    pq_m = _codebooks(codebooks, d)
    if codes.dim() != 2 or codes.shape[1] != pq_m:
        raise ValueError("codes must be [n_codes, pq_m]")
    if probe_ids.dim() != 2 or probe_ids.shape[0] != nq:
        raise ValueError("probe_ids must be [nq, nprobe]")
    if list_offsets.numel() != centroids.shape[0] + 1:
        raise ValueError("list_offsets must have nlist + 1 entries")
    dev = queries.device
    out_ids = torch.empty((nq, n_rerank), dtype=torch.int64, device=dev)
    out_est = torch.empty((nq, n_rerank), dtype=torch.float32, device=dev)
    counts = torch.empty((nq,), dtype=torch.int64, device=dev) if want_counts else None
    with torch.cuda.device(dev):
        rc = lib().ivf_pq_search(_ptr(queries), nq, d, _dtype_code(queries), _ptr(centroids), centroids.shape[0],
                                 _ptr(probe_ids), probe_ids.shape[1], _ptr(list_offsets), _ptr(codes), codes.shape[0],
                                 _ptr(codebooks), pq_m, n_rerank, _ptr(vec_ids), _ptr(out_ids), _ptr(out_est),
                                 _ptr(counts), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)
    return out_ids, out_est, counts


def ivf_centroid_finalize(sums: torch.Tensor, counts: torch.Tensor, centroids: torch.Tensor):
    """centroids[l] = sums[l] / counts[l] in place; lists with count 0 keep their row."""
    _dev(sums, "sums", torch.float32)
    _dev(counts, "counts", torch.int64)
    _dev(centroids, "centroids", torch.float32)
    nlist, d = centroids.shape
    dev = centroids.device
    with torch.cuda.device(dev):
        rc = lib().ivf_centroid_finalize(_ptr(sums), _ptr(counts), nlist, d, _ptr(centroids), _stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_assign_update(points: torch.Tensor, centroids: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor,
                      out_ids: torch.Tensor | None = None, out_dists: torch.Tensor | None = None,
                      chunk_rows: int = 0):
    """One streamed pass of a Lloyd iteration: per chunk copy (if host), assign, accumulate."""
    _rows(points, "points")
    _dev(centroids, "centroids", torch.float32)
    _dev(sums, "sums", torch.float32)
    _dev(counts, "counts", torch.int64)
    n, d = points.shape
    dev = centroids.device
    if out_ids is not None:
        _out(out_ids, "out_ids", torch.int32)
    if out_dists is not None:
        _out(out_dists, "out_dists", torch.float32)
    with torch.cuda.device(dev):
        rc = lib().ivf_assign_update(_ptr(points), n, d, _dtype_code(points), _ptr(centroids), centroids.shape[0],
                                     _ptr(out_ids), _ptr(out_dists), _ptr(sums), _ptr(counts), chunk_rows,
                                     _stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_check(device=None) -> None:
    """Synchronises the current stream and raises if a kernel recorded a device-side problem."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        rc = lib().ivf_check(_stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_launch_count() -> int:
    return int(lib().ivf_launch_count())


def ivf_release_workspace() -> None:
    rc = lib().ivf_release_workspace()
    if rc != IVF_OK:
        _raise(rc)


def ivf_debug_plan(n: int, nlist: int, d: int, k: int, num_sms: int = 148) -> dict:
    out = (ctypes.c_int64 * 9)()
    rc = lib().ivf_debug_plan(n, nlist, d, k, num_sms, out)
    if rc != IVF_OK:
        _raise(rc)
    keys = ("row_tiles", "col_tiles", "ctas", "partials", "block_n", "k_slices", "stages", "smem_bytes", "mtiles")
    return dict(zip(keys, (int(v) for v in out)))


def ivf_debug_span(n: int, nlist: int, d: int, k: int, num_sms: int, cta: int):
    out = (ctypes.c_int64 * 4)()
    rc = lib().ivf_debug_span(n, nlist, d, k, num_sms, cta, out)
    if rc != IVF_OK:
        _raise(rc)
    if int(out[2]) != cta or int(out[3]) != cta:
        raise AssertionError(f"unit-to-CTA mapping disagrees with the span of CTA {cta}: {list(out)}")
    return int(out[0]), int(out[1])


def ivf_debug_rotation(n: int, nlist: int, d: int, k: int, num_sms: int, row_group: int) -> int:
    rc = lib().ivf_debug_rotation(n, nlist, d, k, num_sms, row_group)
    if rc < 0:
        _raise(rc)
    return int(rc)


def ivf_debug_set_threshold_pass(split: bool) -> None:
    lib().ivf_debug_set_threshold_pass(1 if split else 0)


def ivf_debug_set_rotation(on: bool) -> None:
    lib().ivf_debug_set_rotation(1 if on else 0)


def ivf_debug_fail_next_alloc(count: int) -> None:
    lib().ivf_debug_fail_next_alloc(int(count))


def ivf_debug_bounds_checked() -> bool:
    return bool(lib().ivf_debug_bounds_checked())


def ivf_debug_bounds_probe() -> None:
    dev = torch.device("cuda", torch.cuda.current_device())
    rc = lib().ivf_debug_bounds_probe(_stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_debug_set_wait_limit_ns(ns: int) -> None:
    lib().ivf_debug_set_wait_limit_ns(ns)


TIMING_FAMILIES = ("prep", "fused_argmin", "fused_topk", "merge", "update", "threshold_pass",
                   "pq_encode", "pq_scan", "pq_merge")


def ivf_debug_set_crossing_cost(units: int) -> None:
    lib().ivf_debug_set_crossing_cost(int(units))


def ivf_debug_set_dependent_launch(on: bool) -> None:
    lib().ivf_debug_set_dependent_launch(int(on) if not isinstance(on, bool) else (251 if on else 0))


def ivf_debug_set_pq_groups(groups: int) -> None:
    lib().ivf_debug_set_pq_groups(int(groups))


def ivf_debug_timing(enable: bool) -> None:
    lib().ivf_debug_timing(1 if enable else 0)


def ivf_debug_timing_read() -> dict:
    """{family: (milliseconds, launch groups)} since the last read; synchronises the device."""
    ms = (ctypes.c_double * len(TIMING_FAMILIES))()
    cnt = (ctypes.c_int64 * len(TIMING_FAMILIES))()
    rc = lib().ivf_debug_timing_read(ms, cnt)
    if rc != IVF_OK:
        _raise(rc)
    return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(TIMING_FAMILIES)}


def ivf_debug_wait_probe() -> None:
    """Launches the orphaned-wait probe on the current stream (see the header)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    rc = lib().ivf_debug_wait_probe(_stream(dev))
    if rc != IVF_OK:
        _raise(rc)


def ivf_debug_force_fallback(on: bool) -> None:
    lib().ivf_debug_force_fallback(1 if on else 0)


def ivf_debug_rule(k: int, nlist: int):
    """(rule, sample stride): -1 argmin, 0 running, 1 given (threshold pass), 2 bounded."""
    out = (ctypes.c_int * 2)()
    rc = lib().ivf_debug_rule(k, nlist, out)
    if rc != IVF_OK:
        _raise(rc)
    return int(out[0]), int(out[1])


def ivf_debug_stats(enable: bool) -> dict:
    """Counters of the k > 1 path since the last read (see the header); then switches counting on/off."""
    out = (ctypes.c_int64 * 3)()
    rc = lib().ivf_debug_stats(1 if enable else 0, out)
    if rc != IVF_OK:
        _raise(rc)
    return {"selections": int(out[0]), "log_entries": int(out[1]), "fallback_rows": int(out[2])}


def ivf_debug_set_row_chunk(rows: int) -> None:
    lib().ivf_debug_set_row_chunk(rows)
