"""Seeded synthetic inputs shaped like the paper's workloads (Table 2: SIFT-1B is
uint8 with d=128, DEEP-1B is float32 with d=96).

This module only draws inputs.  It holds none of the method's arithmetic (no
distances, no selection, no centroid update), so both the CUDA path's tests and
the CPU oracle's tests may import it without sharing any computation.

Every stream is derived from ``numpy.random.SeedSequence([config_index, stream_id, ...])``
so any chunk of any configuration can be regenerated on its own.

Stream ids
    0  mixture parameters (component means)
    1  centroids
    2  queries
    3  base / training rows (followed by the chunk index)
    4  k-means initialisation sample
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

N_COMPONENTS = 1000
CHUNK_ROWS = 1 << 20  # rows per streamed chunk (Table 3: assignment batch 1,048,576)


@dataclass(frozen=True)
class RoutingConfig:
    """One routing workload: nq queries against nlist centroids, nprobe lists kept."""
    name: str
    index: int
    nq: int
    nlist: int
    d: int
    nprobe: int
    qtype: str  # "f32" or "u8"
    family: str  # "gauss", "sift", "deep"


C0 = RoutingConfig("C0 tiny routing", 0, 1_000, 1_024, 128, 16, "f32", "gauss")
C1 = RoutingConfig("C1 SIFT-shaped routing", 1, 10_000, 65_536, 128, 64, "u8", "sift")
C2 = RoutingConfig("C2 DEEP-shaped routing", 2, 10_000, 262_144, 96, 128, "f32", "deep")
C4 = RoutingConfig("C4 large-batch routing stress", 4, 100_000, 1_048_576, 96, 256, "f32", "deep")
ROUTING_CONFIGS = {0: C0, 1: C1, 2: C2, 4: C4}

# C3: IVF build assignment (streamed Lloyd iterations)
C3_N = 100_000_000
C3_NLIST = 65_536
C3_D = 128
C3_ITERS = 5


def _rng(*key: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence(list(key)))


def _sift_means(family_index: int, d: int) -> np.ndarray:
    # component means U[0,128] per dimension
    return _rng(family_index, 0).uniform(0.0, 128.0, size=(N_COMPONENTS, d)).astype(np.float32)


def _deep_means(family_index: int, d: int) -> np.ndarray:
    # component means N(0,1) per dimension
    return _rng(family_index, 0).standard_normal((N_COMPONENTS, d), dtype=np.float32)


def _mixture_rows(rng: np.random.Generator, means: np.ndarray, rows: int, std: float) -> np.ndarray:
    """rows draws from the uniform-weight Gaussian mixture, float32."""
    comp = rng.integers(0, means.shape[0], size=rows)
    out = rng.standard_normal((rows, means.shape[1]), dtype=np.float32)
    out *= np.float32(std)
    out += means[comp]
    return out


def _to_u8(x: np.ndarray) -> np.ndarray:
    # round half to even, then clip to the byte range
    return np.clip(np.rint(x), 0, 255).astype(np.uint8)


def _unit_rows(x: np.ndarray) -> np.ndarray:
    nrm = np.sqrt((x.astype(np.float64) ** 2).sum(axis=1, keepdims=True))
    nrm[nrm == 0] = 1.0
    return (x / nrm).astype(np.float32)


def sift_like_centroids(nlist: int, d: int = 128, family_index: int = 1) -> np.ndarray:
    """float32 centroids: fresh mixture samples plus N(0, variance 4) noise, unclipped."""
    means = _sift_means(family_index, d)
    rng = _rng(family_index, 1)
    c = _mixture_rows(rng, means, nlist, 20.0)
    c += rng.standard_normal(c.shape, dtype=np.float32) * np.float32(2.0)
    return np.ascontiguousarray(c)


def sift_like_queries(nq: int, d: int = 128, family_index: int = 1) -> np.ndarray:
    means = _sift_means(family_index, d)
    return _to_u8(_mixture_rows(_rng(family_index, 2), means, nq, 20.0))


def sift_like_rows(chunk: int, rows: int = CHUNK_ROWS, d: int = 128, family_index: int = 1,
                   config_index: int = 3) -> np.ndarray:
    """uint8 base rows of one streamed chunk (same mixture as the SIFT-shaped routing case)."""
    means = _sift_means(family_index, d)
    return _to_u8(_mixture_rows(_rng(config_index, 3, chunk), means, rows, 20.0))


def deep_like_centroids(nlist: int, d: int = 96, family_index: int = 2) -> np.ndarray:
    means = _deep_means(family_index, d)
    return _unit_rows(_mixture_rows(_rng(family_index, 1), means, nlist, 0.3))


def deep_like_queries(nq: int, d: int = 96, family_index: int = 2, stream_key: int = 2) -> np.ndarray:
    means = _deep_means(family_index, d)
    return _unit_rows(_mixture_rows(_rng(family_index, stream_key), means, nq, 0.3))


def deep_like_rows(chunk: int, rows: int, d: int = 96, family_index: int = 2) -> np.ndarray:
    """float32 unit-norm base rows of one chunk (DEEP-shaped assignment input)."""
    means = _deep_means(family_index, d)
    return _unit_rows(_mixture_rows(_rng(family_index, 3, chunk), means, rows, 0.3))


def routing_inputs(cfg: RoutingConfig, nq: int | None = None, nlist: int | None = None):
    """(queries, centroids) of a routing configuration; nq/nlist may be cut down for tests
    (a prefix of the same seeded streams is NOT guaranteed, the draw is simply smaller)."""
    nq = cfg.nq if nq is None else nq
    nlist = cfg.nlist if nlist is None else nlist
    if cfg.family == "gauss":
        rng = _rng(0)
        q = rng.standard_normal((nq, cfg.d), dtype=np.float32)
        c = rng.standard_normal((nlist, cfg.d), dtype=np.float32)
        return q, c
    if cfg.family == "sift":
        return sift_like_queries(nq, cfg.d, 1), sift_like_centroids(nlist, cfg.d, 1)
    if cfg.family == "deep":
        return deep_like_queries(nq, cfg.d, 2), deep_like_centroids(nlist, cfg.d, 2)
    raise ValueError(cfg.family)


def init_sample(n: int, nlist: int, config_index: int = 3) -> np.ndarray:
    """Sorted row indices of the uniform sample without replacement that seeds k-means."""
    idx = _rng(config_index, 4).choice(n, size=nlist, replace=False)
    idx.sort()
    return idx.astype(np.int64)


def integer_case(nq: int, nlist: int, d: int, seed: int, hi: int = 256):
    """uint8 queries and integer-valued float32 centroids in [0, hi): every product and sum is an
    exact small integer in fp16, fp32 and fp64 alike, and ties are plentiful."""
    rng = _rng(99, seed)
    q = rng.integers(0, hi, size=(nq, d)).astype(np.uint8)
    c = rng.integers(0, hi, size=(nlist, d)).astype(np.float32)
    return q, c


# ------------------------------------------------------------------ residual-PQ inputs (stream ids 5-8)
def pq_codebooks(pq_m: int, dsub: int, scale: float, seed: int, integer: bool = False) -> np.ndarray:
    """float32 [pq_m, 256, dsub] codebooks: i.i.d. N(0, scale^2) entries (rounded to integers on
    request).  A stand-in for trained codebooks with the spread of the residuals they quantise."""
    cb = _rng(5, seed).normal(0.0, scale, size=(pq_m, 256, dsub))
    if integer:
        cb = np.rint(cb)
    return cb.astype(np.float32)


def skewed_list_ids(n: int, nlist: int, seed: int, sigma: float = 1.0):
    """(ids int32 [n] in list-major (sorted) order, offsets int64 [nlist + 1]): list lengths drawn
    from a multinomial with log-normal weights, so they vary by more than an order of magnitude
    and some lists may be empty, as inverted lists do."""
    rng = _rng(6, seed)
    w = rng.lognormal(0.0, sigma, size=nlist)
    counts = rng.multinomial(n, w / w.sum())
    offsets = np.zeros(nlist + 1, np.int64)
    np.cumsum(counts, out=offsets[1:])
    ids = np.repeat(np.arange(nlist, dtype=np.int32), counts)
    return ids, offsets


def rows_near(c: np.ndarray, ids: np.ndarray, noise_std: float, seed: int, dtype: str = "f32") -> np.ndarray:
    """Rows drawn around given centroid rows: c[ids] + N(0, noise_std^2); 'u8' rounds and clips."""
    rng = _rng(7, seed)
    x = c[ids] + rng.normal(0.0, noise_std, size=(len(ids), c.shape[1])).astype(np.float32)
    return _to_u8(x) if dtype == "u8" else x.astype(np.float32)


def distinct_probes(nq: int, nlist: int, nprobe: int, seed: int) -> np.ndarray:
    """int32 [nq, nprobe]: nprobe distinct list ids per query, uniformly drawn, in random order."""
    rng = _rng(8, seed)
    out = np.empty((nq, nprobe), np.int32)
    for b in range(nq):
        out[b] = rng.choice(nlist, size=nprobe, replace=False)
    return out


# ------------------------------------------------------------------ SPACEV-shaped inputs (Table 2: int8, d = 100)
def spacev_like(rows: int, nlist: int, seed: int, d: int = 100):
    """(points int8 [rows, d], centroids float32 [nlist, d]): a 1,000-component mixture (means
    N(0, 30^2), std 12) rounded and clipped to signed bytes; centroids are fresh mixture samples
    with N(0, 1) noise, unrounded."""
    rng = _rng(9, seed)
    means = rng.normal(0.0, 30.0, size=(N_COMPONENTS, d)).astype(np.float32)
    x = _mixture_rows(rng, means, rows, 12.0)
    c = _mixture_rows(rng, means, nlist, 12.0) + rng.normal(0.0, 1.0, size=(nlist, d)).astype(np.float32)
    return np.clip(np.rint(x), -128, 127).astype(np.int8), c.astype(np.float32)
