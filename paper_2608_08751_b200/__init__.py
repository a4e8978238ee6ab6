"""B200-native IVF routing / assignment hot path (squared-L2 distance to every centroid with a
fused per-row top-k, plus the Lloyd centroid update).  The compute lives in the C-ABI library
built from ``csrc/``; ``binding`` marshals arguments and nothing else."""

__all__ = ["binding", "synth"]
