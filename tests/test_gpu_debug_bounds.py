"""The bounds-checked build of the library (-DCCR_DEBUG_BOUNDS): every global address the join kernels compute is
checked against the extents of the launch's buffers; an address outside is skipped (never a trap) and reported as
CCR_ERR_BOUNDS.  compute-sanitizer is not available where these tests run, so this build is the stand-in for it:
the tiny, random, boundary and non-uniform-key parity tests are run once more against it in a child process (their
own checks include a clean device status, so any flagged address fails them), and the mechanism itself is shown to
fire by registering output extents that end one row early."""
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2609_22441_b200 import workloads as W

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def debug_lib():
    from paper_2609_22441_b200 import build

    return build.build_debug()


def test_parity_suites_run_clean_under_the_bounds_checked_build(debug_lib):
    env = dict(os.environ, CCR_LIB_OVERRIDE=debug_lib)
    out = subprocess.run(
        [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "tests/test_gpu_random.py", "tests/test_gpu_parity.py",
         "tests/test_gpu_padded.py", "-k",
         "tiny or random or boundaries or generic or holes or all_found or many_small or worked or (clustered and 37) or unresolved"],
        cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout


def test_an_address_outside_the_buffers_is_skipped_and_reported(debug_lib):
    code = r"""
import numpy as np, torch, sys
from paper_2609_22441_b200 import binding as B, workloads as W
assert B.lib().ccr_debug_bounds_enabled() == 1
for flags in (B.CCR_FLAG_WARP_SPECIALISED, B.CCR_FLAG_TWO_PHASE):
    wl = W.config1(n_docs=20_000, n_req=3, n_cand=700)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    n, out_b = db.total_cands, store.out_row_bytes()
    rows = torch.full((n, out_b), 0xA5, dtype=torch.uint8, device="cuda")
    mask = torch.full((n,), 0xA5, dtype=torch.uint8, device="cuda")
    good_rows, good_mask = B.join_batch(store, db, flags)
    assert store.device_status() == B.CCR_OK
    B.lib().ccr_debug_shrink_outputs(store.handle, 1)          # the registered outputs end one row early
    B.join_batch(store, db, flags, rows, mask)
    assert store.device_status() == B.CCR_ERR_BOUNDS           # reported ...
    assert store.device_status() == B.CCR_OK                   # ... once
    assert torch.equal(rows[:-1], good_rows[:-1]) and torch.equal(mask[:-1], good_mask[:-1])
    assert (rows[-1] == 0xA5).all() and mask[-1] == 0xA5       # the stores to the last row were left out
    B.lib().ccr_debug_shrink_outputs(store.handle, 0)
    B.join_batch(store, db, flags, rows, mask)
    assert store.device_status() == B.CCR_OK and torch.equal(rows, good_rows)
    store.free()
print("ok")
"""
    env = dict(os.environ, CCR_LIB_OVERRIDE=debug_lib)
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout[-2000:] + out.stderr[-3000:]


def test_release_build_has_no_checks():
    from paper_2609_22441_b200 import binding as B

    assert B.lib().ccr_debug_bounds_enabled() == 0
