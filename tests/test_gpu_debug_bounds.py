"""The bounds-checked build of the library (-DCCR_DEBUG_BOUNDS): every global address the join, sort, resolve,
compaction and upsert kernels compute is checked against the extents of the launch's buffers; an address outside is
skipped (never a trap) and reported as CCR_ERR_BOUNDS (by ccr_docstore_device_status for the joins, as the call's own
status for the others, which this build runs synchronously).  compute-sanitizer is not available where these tests run, so this build is the stand-in for it:
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


def test_sort_resolve_compaction_and_upsert_run_clean_under_the_bounds_checked_build(debug_lib):
    """In this build those calls wait for their kernels and return CCR_ERR_BOUNDS themselves, so the binding raises
    on any flagged address."""
    env = dict(os.environ, CCR_LIB_OVERRIDE=debug_lib)
    out = subprocess.run(
        [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "tests/test_gpu_sort.py", "tests/test_gpu_resolve.py",
         "tests/test_gpu_upsert.py", "tests/test_gpu_pipeline.py", "tests/test_gpu_padded.py", "-k",
         "not more_row_tiles and not hundred_million and not full_size"],
        cwd=ROOT, env=env, capture_output=True, text=True, timeout=2400)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout


def test_a_sort_whose_output_rows_end_early_is_reported_and_skips_the_row(debug_lib):
    code = r"""
import numpy as np, torch
from oracle import oracle
from paper_2609_22441_b200 import binding as B, workloads as W
assert B.lib().ccr_debug_bounds_enabled() == 1
rng = np.random.default_rng(5)
lens = [5000, 9000, 100, 0, 4097]
keys = rng.integers(0, 1 << 30, size=sum(lens), dtype=np.int64)
feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
want_k, want_f, want_p = oracle.sort_edges(keys, feats, eo)
wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
store = B.store_from_workload(wl)
dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
k_in, f_in, o = dev(keys), dev(feats), dev(eo)
def run():
    k = torch.full((len(keys),), -7, dtype=torch.int64, device="cuda")
    f = torch.full(feats.shape, 7.0, dtype=torch.float16, device="cuda")
    p = torch.full((len(keys),), -7, dtype=torch.int32, device="cuda")
    try:
        B.ccr_sort_edges(store, len(lens), max(lens), k_in, f_in, o, k, f, p)
        st = B.CCR_OK
    except B.CcrError as e:
        st = e.status
    torch.cuda.synchronize()
    return st, k.cpu().numpy(), f.cpu().numpy(), p.cpu().numpy()
st, k, f, p = run()
assert st == B.CCR_OK and np.array_equal(k, want_k) and np.array_equal(p, want_p) and np.array_equal(f.view(np.uint16), want_f.view(np.uint16))
B.lib().ccr_debug_shrink_outputs(store.handle, 1)          # the registered output rows end one row early
st, k, f, p = run()
assert st == B.CCR_ERR_BOUNDS
assert np.array_equal(k, want_k) and np.array_equal(p, want_p)
assert np.array_equal(f[:-1].view(np.uint16), want_f[:-1].view(np.uint16)) and (f[-1] == 7.0).all()
B.lib().ccr_debug_shrink_outputs(store.handle, 0)
st, k, f, p = run()
assert st == B.CCR_OK and np.array_equal(f.view(np.uint16), want_f.view(np.uint16))
store.free()
print("ok")
"""
    env = dict(os.environ, CCR_LIB_OVERRIDE=debug_lib)
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout[-2000:] + out.stderr[-3000:]


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
