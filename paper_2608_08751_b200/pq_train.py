"""Residual-PQ codebook training composed from the library's calls (Sec. 2.2 Eq. 3 learns one
codebook per subspace; Sec. 4.3 trains them on the residuals x - c(x)).

Per subspace this is Lloyd's algorithm with 256 lists on the d / pq_m wide sub-vectors of the
residuals: the same assignment (`ivf_assign_update`) and mean (`ivf_centroid_finalize`) kernels
as the IVF build, at a different shape.  torch is used only to slice a column block of the
residual matrix into a contiguous buffer and to pick the seeded initial codewords; every
distance, arg-min, sum and mean runs in the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding as B


def train_codebooks(points: torch.Tensor, ids: torch.Tensor, centroids: torch.Tensor, pq_m: int, iters: int = 5,
                    seed: int = 0, sample_rows: int | None = None):
    """(codebooks float32 [pq_m, 256, d // pq_m], inertia [pq_m, iters]): k-means per subspace on the
    residuals of `points` (row i assigned to list ids[i]).  `sample_rows` trains on a seeded sample."""
    n, d = points.shape
    if d % pq_m != 0:
        raise ValueError("pq_m must divide d")
    dsub = d // pq_m
    wide = (dsub + 3) // 4 * 4  # the assignment kernel takes rows of 4k floats: zero columns change no distance
    dev = points.device
    gen = torch.Generator(device="cpu").manual_seed(seed)
    if sample_rows is not None and sample_rows < n:
        pick = torch.randperm(n, generator=gen)[:sample_rows].sort().values.to(dev)
        points, ids = points[pick].contiguous(), ids[pick].contiguous()
        n = sample_rows
    if n < 256:
        raise ValueError("at least 256 training rows are needed")
    res = B.ivf_pq_residuals(points, ids, centroids)
    init = torch.randperm(n, generator=gen)[:256].sort().values.to(dev)
    codebooks = torch.empty((pq_m, 256, dsub), dtype=torch.float32, device=dev)
    inertia = torch.zeros((pq_m, iters), dtype=torch.float64)
    sums = torch.empty((256, wide), dtype=torch.float32, device=dev)
    counts = torch.empty((256,), dtype=torch.int64, device=dev)
    a_ids = torch.empty((n,), dtype=torch.int32, device=dev)
    a_d = torch.empty((n,), dtype=torch.float32, device=dev)
    for m in range(pq_m):
        sub = torch.zeros((n, wide), dtype=torch.float32, device=dev)
        sub[:, :dsub] = res[:, m * dsub:(m + 1) * dsub]
        cb = sub[init].clone()
        for it in range(iters):
            sums.zero_()
            counts.zero_()
            B.ivf_assign_update(sub, cb, sums, counts, a_ids, a_d)
            B.ivf_centroid_finalize(sums, counts, cb)
            inertia[m, it] = float(a_d.double().sum().item())
        codebooks[m] = cb[:, :dsub]
    return codebooks, inertia
