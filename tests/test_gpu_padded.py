"""GPU parity of the padded batch layout (Section 6.3.1, batching and padding): ccr_compact_valid followed by
ccr_join_batch_padded, through the C ABI, against the oracle's three-step restatement — every byte of
T[b, n_max, row], the mask, the per-request counts and the kept candidates' source indices."""
import os

import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

from helpers import GUARD, tiny_workload

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def B():
    from paper_2609_22441_b200 import binding, build

    build.build()
    binding.lib()
    return binding


def _oracle_padded(wl, n_max=None, first_degree_only=False):
    s, b = wl.store, wl.batch
    return oracle.join_padded(
        s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets, n_max=n_max,
        req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types, reduce_sum_mask=s.reduce_sum_mask,
        first_degree_only=first_degree_only, n_threads=4)


def _gpu_padded(B, store, db, n_max, flags=0):
    """compact + padded join into guarded, poisoned buffers; returns numpy (T, M, offsets, src)."""
    dev = torch.device("cuda", store.device)
    out_b = store.out_row_bytes(flags)
    n, C = db.n_req * n_max, db.total_cands
    rows_buf = torch.full((GUARD + n * out_b + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
    mask_buf = torch.full((GUARD + n + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
    idx = torch.full((C + 64,), -7, dtype=torch.int32, device=dev)
    src = torch.full((C + 64,), -7, dtype=torch.int32, device=dev)
    offs = torch.full((db.n_req + 1 + 8,), -7, dtype=torch.int64, device=dev)
    B.ccr_compact_valid(store, db.n_req, C, db.cand_idx, db.cand_offsets, idx, offs, src)
    B.ccr_join_batch_padded(store, db.n_req, C, db.max_edge_len, n_max, db.edge_keys, db.edge_feats, db.edge_offsets,
                            idx, offs, db.req_feats, rows_buf[GUARD:], mask_buf[GUARD:], flags)
    torch.cuda.synchronize(dev)
    rb, mb = rows_buf.cpu().numpy(), mask_buf.cpu().numpy()
    assert (rb[:GUARD] == 0xA5).all() and (rb[GUARD + n * out_b:] == 0xA5).all(), "write outside out_rows"
    assert (mb[:GUARD] == 0xA5).all() and (mb[GUARD + n:] == 0xA5).all(), "write outside out_mask"
    offs_h, idx_h, src_h = offs.cpu().numpy(), idx.cpu().numpy(), src.cpu().numpy()
    assert (offs_h[db.n_req + 1:] == -7).all()
    V = int(offs_h[db.n_req]) if db.n_req else 0
    assert (idx_h[V:] == -7).all() and (src_h[V:] == -7).all(), "compaction wrote behind the last valid candidate"
    return (rb[GUARD:GUARD + n * out_b].reshape(db.n_req, n_max, out_b), mb[GUARD:GUARD + n].reshape(db.n_req, n_max),
            offs_h[:db.n_req + 1], src_h[:V], idx_h[:V])


def _check(B, wl, flag_sets=(("ws", 0),), n_max_list=(None,), first_degree_only=False, tunings=((0, 0),)):
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    try:
        for n_max in n_max_list:
            want_T, want_M, n_valid, want_src = _oracle_padded(wl, n_max, first_degree_only)
            nm = want_T.shape[1]
            if nm == 0:
                continue  # nothing valid in the whole batch and no n_max given: the call needs n_max > 0
            for tuning in tunings:
                if any(tuning):
                    store.set_tuning(*tuning)
                for name, flags in flag_sets:
                    if first_degree_only:
                        flags |= B.CCR_FLAG_FIRST_DEGREE_ONLY
                    T, M, offs, src, idx = _gpu_padded(B, store, db, nm, flags)
                    assert np.array_equal(np.diff(offs), n_valid) and offs[0] == 0, (wl.name, name)
                    assert np.array_equal(src, want_src), (wl.name, name)
                    assert np.array_equal(idx, wl.batch.cand_idx[want_src]), (wl.name, name)
                    assert np.array_equal(M, want_M), (wl.name, name, n_max)
                    if not np.array_equal(T, want_T):
                        bad = np.argwhere((T != want_T).any(axis=2))
                        raise AssertionError("%s/%s n_max=%s: %d slots differ, first %s" %
                                             (wl.name, name, n_max, len(bad), bad[0]))
        assert store.device_status() == B.CCR_OK
    finally:
        store.free()


def _kernels(B):
    return [("ws", 0), ("ws+static", B.CCR_FLAG_STATIC_SPLIT), ("2phase", B.CCR_FLAG_TWO_PHASE),
            ("ws+global", B.CCR_FLAG_FORCE_GLOBAL), ("2phase+sampled", B.CCR_FLAG_TWO_PHASE | B.CCR_FLAG_FORCE_SAMPLED)]


def test_worked_example_of_the_paper(B):
    """R0 = [10, 42, 87], R1 = [5, 63] -> T[0] = f10 f42 f87, T[1] = f5 f63 pad."""
    req = [[int(x) for x in line.split(":")[1].split()]
           for line in open(os.path.join(GOLDEN, "batching_example.txt")) if line.startswith("request")]
    rng = np.random.default_rng(1)
    store_h = W.make_store(rng, 100, 50, 8, np.float32, tagged=True)
    keys, feats = W.make_viewer(rng, 50, 5, 8, np.float16)
    batch = W.assemble_batch([keys, keys], [feats, feats], [np.array(x, np.int32) for x in req], None, 8, np.float16, 0,
                             np.float32)
    wl = W.Workload("example", 1, store_h, batch)
    store = B.store_from_workload(wl)
    try:
        T, M, offs, src, idx = _gpu_padded(B, store, B.DeviceBatch(batch), 3)
    finally:
        store.free()
    assert list(offs) == [0, 3, 5] and list(idx) == [10, 42, 87, 5, 63] and list(src) == [0, 1, 2, 3, 4]
    first = T[:, :, :4].copy().view(np.float32)[:, :, 0]  # tagged store: row p starts with p * 8
    assert first.tolist() == [[80.0, 336.0, 696.0], [40.0, 504.0, 0.0]]
    assert not T[1, 2].any() and M[1, 2] == 0
    _check(B, wl, _kernels(B), n_max_list=(None, 7, 2))


@pytest.mark.parametrize("seed", range(12))
def test_tiny_batches_with_unresolved_positions(B, seed):
    rng = np.random.default_rng(seed)
    second = bool(seed & 1)
    wl = tiny_workload(1000 + seed, int(rng.integers(1, 60)), int(rng.integers(1, 30)), int(rng.integers(1, 6)), 16,
                       int(rng.integers(1, 90)), second, 4 if seed % 3 == 0 else 0)
    _check(B, wl, _kernels(B), n_max_list=(None, 100, 3), tunings=((0, 0), (512, 0, 3, 2, 1)))
    if second:
        _check(B, wl, [("ws", 0), ("2phase", B.CCR_FLAG_TWO_PHASE)], first_degree_only=True)


def _with_unresolved(wl, frac, seed):
    """Replace a fraction of the positions by -1 (unknown id) or n_docs (out of range)."""
    rng = np.random.default_rng(seed)
    ci = wl.batch.cand_idx.copy()
    hit = rng.random(len(ci)) < frac
    ci[hit] = np.where(rng.random(int(hit.sum())) < 0.8, -1, wl.store.n_docs).astype(np.int32)
    wl.batch.cand_idx = ci
    return wl


def test_ragged_multi_tile_batch(B):
    """Requests of very different lengths (so most of T is pads for some), several tiles each, a ragged tail,
    empty requests, 15 % unresolved positions."""
    base = W.config1(n_docs=60_000, n_req=7, n_cand=5_000)
    s, b = base.store, base.batch
    lens = [5_000, 0, 37, 2_049, 1, 0, 4_999]
    keys_l, feats_l, cands_l = [], [], []
    for r, n in enumerate(lens):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0 = int(b.cand_offsets[r])
        keys_l.append(b.edge_keys[e0:e1])
        feats_l.append(b.edge_feats[e0:e1])
        cands_l.append(b.cand_idx[c0:c0 + n])
    batch = W.assemble_batch(keys_l, feats_l, cands_l, b.req_feats, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype)
    wl = _with_unresolved(W.Workload("ragged", 5, s, batch), 0.15, 11)
    _check(B, wl, _kernels(B), n_max_list=(None, 6_000, 1_000), tunings=((0, 0), (512, 0, 5, 3, 2)))


def test_many_small_requests(B):
    """1500 requests (more than the kernels mirror in shared memory, several rounds of the offset scan)."""
    wl = _with_unresolved(W.config1(n_docs=30_000, n_req=1500, n_cand=150, edge_lo=3, edge_hi=80), 0.2, 4)
    _check(B, wl, [("ws", 0), ("2phase", B.CCR_FLAG_TWO_PHASE)], n_max_list=(None, 40))


def test_sorted_candidates_take_the_merge_path(B):
    """Compaction keeps the input order, so candidates sorted by author id stay sorted."""
    wl = W.sort_candidates_by_author(W.config1(n_docs=50_000, n_req=5, n_cand=4_000))
    _check(B, wl, [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])


def test_second_degree_scaled(B):
    wl = _with_unresolved(W.config1(n_docs=50_000, n_req=4, n_cand=3_000, second_degree=True), 0.1, 3)
    _check(B, wl, [("ws", 0), ("2phase", B.CCR_FLAG_TWO_PHASE)])


def test_all_unresolved_and_argument_errors(B):
    wl = tiny_workload(5, 20, 10, 3, 8, 40, False, 0)
    wl.batch.cand_idx = np.full_like(wl.batch.cand_idx, -1)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    try:
        T, M, offs, src, idx = _gpu_padded(B, store, db, 4)
        assert not T.any() and not M.any() and not offs.any() and len(src) == 0
        L = B.lib()
        assert L.ccr_join_batch_padded(store.handle, 1, 1, 1, 0, None, None, None, None, None, None, None, None, 0,
                                       None) == B.CCR_ERR_INVALID_ARG
        assert L.ccr_join_batch_padded(store.handle, 1, 1, 1, 4, None, None, None, None, None, None, None, None,
                                       B.CCR_FLAG_VALIDATE, None) == B.CCR_ERR_UNSUPPORTED
        assert L.ccr_compact_valid(store.handle, -1, 0, None, None, None, None, None, None) == B.CCR_ERR_INVALID_ARG
        assert L.ccr_compact_valid(store.handle, 0, 0, None, None, None, None, None, None) == B.CCR_OK
        assert L.ccr_compact_valid(store.handle, 1, 0, None, None, None, None, None, None) == B.CCR_ERR_INVALID_ARG
        assert store.device_status() == B.CCR_OK
    finally:
        store.free()


def test_config1_full_size_padded_equals_ragged_rows_in_place(B):
    """At the benchmark's full size (64 x 30,000 candidates, 1M docs), in its launch configuration: T is the
    ragged join's output (checked against the oracle elsewhere) re-addressed — T[r, :n_r] equals rows
    [offsets[r], offsets[r+1]) of ccr_join_batch over the compacted batch, everything behind is zero — and
    sampled slots are recomputed by the oracle one by one."""
    wl = _with_unresolved(W.config1(), 0.05, 21)
    s, b = wl.store, wl.batch
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(b)
    try:
        T, M, offs, src = B.join_batch_padded(store, db)
        torch.cuda.synchronize()
        n_max = T.shape[1]
        assert n_max == 30_000
        offs_h = offs.cpu().numpy()
        V = int(offs_h[-1])
        src_h = src[:V].cpu().numpy()
        valid = (b.cand_idx >= 0) & (b.cand_idx < s.n_docs)
        assert np.array_equal(src_h, np.nonzero(valid)[0])
        assert np.array_equal(np.diff(offs_h), np.add.reduceat(valid, b.cand_offsets[:-1]))
        # ragged join over the compacted candidates
        cdb = B.DeviceBatch(b)
        cdb.cand_idx = torch.from_numpy(b.cand_idx[valid]).cuda()
        cdb.cand_offsets = offs
        cdb.total_cands = V
        rows, mask = B.join_batch(store, cdb)
        torch.cuda.synchronize()
        for r in range(b.n_req):
            c0, c1 = int(offs_h[r]), int(offs_h[r + 1])
            assert torch.equal(T[r, :c1 - c0], rows[c0:c1]) and torch.equal(M[r, :c1 - c0], mask[c0:c1])
            assert not T[r, c1 - c0:].any() and not M[r, c1 - c0:].any()
        # sampled slots against the oracle: candidates src[k] of the original batch
        rng = np.random.default_rng(2)
        ks = np.unique(np.concatenate([rng.integers(0, V, size=4_000), offs_h[:-1], offs_h[1:] - 1]))
        J = src_h[ks].astype(np.int64)
        req_of = np.searchsorted(b.cand_offsets, J, side="right") - 1
        co = np.searchsorted(req_of, np.arange(b.n_req + 1), side="left").astype(np.int64)
        want_rows, want_mask = oracle.join(s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets,
                                           b.cand_idx[J], co, req_feats=b.req_feats, n_threads=4)
        slot = ks - offs_h[req_of]
        got = T[torch.from_numpy(req_of).cuda(), torch.from_numpy(slot).cuda()].cpu().numpy()
        gotm = M[torch.from_numpy(req_of).cuda(), torch.from_numpy(slot).cuda()].cpu().numpy()
        assert np.array_equal(got, want_rows) and np.array_equal(gotm, want_mask)
        assert store.device_status() == B.CCR_OK
    finally:
        store.free()
