"""Builds the C-ABI library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Two variants: the regular library, and a checked one (-DIVF_CHECK_BOUNDS) whose kernels verify their
shared-memory, tensor-memory and global indices and report the first violation through the status
word instead of touching memory out of range -- selected at load time with IVF_B200_CHECKED=1."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libivf_b200.so")
CHECKED_LIB_PATH = os.path.join(_PKG, "libivf_b200_checked.so")
_SOURCES = ["ivf_api.cu"]
_HEADERS = ["ptx.cuh", "check.cuh", "scales.cuh", "fused_topk.cuh", "merge.cuh", "prep.cuh", "update.cuh", "pq.cuh",
            "candidates.cuh"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    deps = [os.path.join(_CSRC, f) for f in _SOURCES + _HEADERS] + [os.path.join(_ROOT, "include", "ivf_b200.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    out = CHECKED_LIB_PATH if checked else LIB_PATH
    if not force and not _stale(out):
        return out
    tmp = out + f".{os.getpid()}.tmp"
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include")]
    if checked:
        cmd += ["-DIVF_CHECK_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(_CSRC, s) for s in _SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
