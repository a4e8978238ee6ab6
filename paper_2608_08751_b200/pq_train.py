"""Residual-PQ codebook training composed from the library's calls (Sec. 2.2 Eq. 3 learns one
codebook per subspace; Sec. 4.3 trains them on the residuals x - c(x)).

Per subspace this is Lloyd's algorithm with 256 lists on the d / pq_m wide sub-vectors of the
residuals.  The assignment step of all subspaces at once is exactly the encoder
(`ivf_pq_encode`: the nearest codeword per subspace); the update step is the IVF build's
sum/count kernel and mean (`ivf_centroid_update`, `ivf_centroid_finalize`) on each sub-vector
block with the code bytes as list ids.  torch is used only to slice a column block of the
residual matrix into a contiguous, zero-padded buffer, to widen the code bytes to int32 and to
pick the seeded initial codewords; every distance, arg-min, sum and mean runs in the library's
kernels.  `method="assign"` runs the assignment through `ivf_assign_update` instead (the tensor-core
kernel at a 256-list, sub-vector-wide shape: slower, but it also returns the inertia).
"""
from __future__ import annotations

import torch

from . import binding as B


def train_codebooks(points: torch.Tensor, ids: torch.Tensor, centroids: torch.Tensor, pq_m: int, iters: int = 5,
                    seed: int = 0, sample_rows: int | None = None, method: str = "encode"):
    """(codebooks float32 [pq_m, 256, d // pq_m], inertia [pq_m, iters] or None): k-means per subspace
    on the residuals of `points` (row i assigned to list ids[i]).  `sample_rows` trains on a seeded
    sample.  The inertia (summed squared distance per subspace and iteration) is only available with
    method="assign"."""
    n, d = points.shape
    if d % pq_m != 0:
        raise ValueError("pq_m must divide d")
    if method not in ("encode", "assign"):
        raise ValueError("method must be 'encode' or 'assign'")
    dsub = d // pq_m
    wide = (dsub + 3) // 4 * 4  # the update / assignment kernels take rows of 4k floats: zero columns change nothing
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
    sums = torch.empty((256, wide), dtype=torch.float32, device=dev)
    counts = torch.empty((256,), dtype=torch.int64, device=dev)

    def block(m):  # contiguous, zero-padded copy of subspace m's columns
        sub = torch.zeros((n, wide), dtype=torch.float32, device=dev)
        sub[:, :dsub] = res[:, m * dsub:(m + 1) * dsub]
        return sub

    if method == "assign":
        codebooks = torch.empty((pq_m, 256, dsub), dtype=torch.float32, device=dev)
        inertia = torch.zeros((pq_m, iters), dtype=torch.float64)
        a_ids = torch.empty((n,), dtype=torch.int32, device=dev)
        a_d = torch.empty((n,), dtype=torch.float32, device=dev)
        for m in range(pq_m):
            sub = block(m)
            cb = sub[init].clone()
            for it in range(iters):
                sums.zero_()
                counts.zero_()
                B.ivf_assign_update(sub, cb, sums, counts, a_ids, a_d)
                B.ivf_centroid_finalize(sums, counts, cb)
                inertia[m, it] = float(a_d.double().sum().item())
            codebooks[m] = cb[:, :dsub]
        return codebooks, inertia

    wide_cb = torch.zeros((pq_m, 256, wide), dtype=torch.float32, device=dev)
    for m in range(pq_m):
        wide_cb[m, :, :dsub] = res[init, m * dsub:(m + 1) * dsub]
    for _ in range(iters):
        codes = B.ivf_pq_encode(points, ids, centroids, wide_cb[:, :, :dsub].contiguous())
        for m in range(pq_m):
            sums.zero_()
            counts.zero_()
            B.ivf_centroid_update(block(m), codes[:, m].to(torch.int32).contiguous(), sums, counts)
            B.ivf_centroid_finalize(sums, counts, wide_cb[m])
    return wide_cb[:, :, :dsub].contiguous(), None
