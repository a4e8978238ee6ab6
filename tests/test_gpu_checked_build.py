"""The checked build (-DIVF_CHECK_BOUNDS) and the allocation-failure hook.

No memory checker can be run on the GPU machines this library is tested on, so the library carries
its own: a second build whose kernels verify their shared-memory, tensor-memory and global indices,
record the first violation in the status word and skip the access.  Here the small-case, random-shape
and PQ parity suites are run once more in a child process that loads that build (IVF_B200_CHECKED=1);
every one of those tests reads the status word through ivf_check, so a violation fails it."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2608_08751_b200 import binding as B
from paper_2608_08751_b200 import build as libbuild

import parity

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _child(code_or_args, is_pytest):
    env = dict(os.environ, IVF_B200_CHECKED="1")
    cmd = [sys.executable, "-m", "pytest"] + code_or_args if is_pytest else [sys.executable, "-c", code_or_args]
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_checked_build_reports_a_violation_and_the_context_survives():
    libbuild.build(checked=True)
    code = (
        "import numpy as np, torch\n"
        "from paper_2608_08751_b200 import binding as B\n"
        "assert B.ivf_debug_bounds_checked()\n"
        "B.ivf_debug_bounds_probe()\n"
        "try:\n"
        "    B.ivf_check()\n"
        "    raise SystemExit('no violation reported')\n"
        "except B.IvfError as e:\n"
        "    assert e.code == B.IVF_ERR_BOUNDS and 'site 999' in str(e) and 'index 5' in str(e), str(e)\n"
        "B.ivf_check()\n"
        "x = torch.randn(300, 64, device='cuda'); c = torch.randn(900, 64, device='cuda')\n"
        "ids, d = B.ivf_route(x, c, 5)\n"
        "B.ivf_check()\n"
        "ref = torch.cdist(x.double(), c.double()).pow(2).topk(5, largest=False).indices\n"
        "assert (ids.long() == ref).float().mean() > 0.99\n"
        "print('ok')\n")
    r = _child(code, False)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
    assert not B.ivf_debug_bounds_checked()  # this process runs the regular build
    B.ivf_debug_bounds_probe()               # ... where the probe is a no-op
    B.ivf_check()


def test_parity_suites_run_clean_under_the_checked_build():
    libbuild.build(checked=True)
    r = _child(["tests/test_gpu_parity.py", "tests/test_gpu_fuzz.py", "tests/test_gpu_pq.py", "tests/test_gpu_variants.py",
                "tests/test_gpu_candidates.py", "tests/test_gpu_shards.py", "-m", "gpu", "-x", "-q",
                "-k", "not full_size and not config3 and not config4 and not expired_wait and not full_configuration"],
               True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]


def test_refused_workspace_allocation_is_reported_and_the_next_call_works():
    rng = np.random.default_rng(8)
    x = rng.integers(0, 256, (700, 128)).astype(np.uint8)
    c = (rng.standard_normal((5000, 128)) * 40 + 100).astype(np.float32)
    xt, ct = torch.from_numpy(x).cuda(), torch.from_numpy(c).cuda()
    B.ivf_route(xt, ct, 20)
    B.ivf_check()
    B.ivf_release_workspace()          # the next call has to allocate its workspace again
    B.ivf_debug_fail_next_alloc(1)
    try:
        with pytest.raises(B.IvfError) as e:
            B.ivf_route(xt, ct, 20)
        assert e.value.code == B.IVF_ERR_ALLOC and "refused" in str(e.value)
    finally:
        B.ivf_debug_fail_next_alloc(0)
    B.ivf_check()
    ids, dists = B.ivf_route(xt, ct, 20)   # the same call now succeeds
    B.ivf_check()
    parity.check_route(x, c, 20, ids.cpu().numpy(), dists.cpu().numpy())
    # a refusal in the middle of a call (the third allocation) leaves nothing half-done either
    B.ivf_release_workspace()
    B.ivf_debug_fail_next_alloc(0)
    sums = torch.zeros((5000, 128), dtype=torch.float32, device="cuda")
    counts = torch.zeros((5000,), dtype=torch.int64, device="cuda")
    a_ids = torch.empty((700,), dtype=torch.int32, device="cuda")
    B.ivf_assign(xt, ct, a_ids, None, want_dists=False)
    B.ivf_check()
    B.ivf_release_workspace()
    B.ivf_debug_fail_next_alloc(1)
    with pytest.raises(B.IvfError) as e:
        B.ivf_centroid_update(xt, a_ids, sums, counts)
    assert e.value.code == B.IVF_ERR_ALLOC
    B.ivf_check()
    assert counts.sum().item() == 0      # nothing was accumulated by the refused call
    B.ivf_centroid_update(xt, a_ids, sums, counts)
    B.ivf_check()
    parity.check_update(x, a_ids.cpu().numpy(), 5000, sums.cpu().numpy(), counts.cpu().numpy())
