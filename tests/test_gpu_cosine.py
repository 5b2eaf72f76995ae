"""GPU parity of the derived cosine section (Section 4.1.2: per-medoid chunked cosine similarity, float32 math,
float16 result) computed inside the join kernel, through ccr_join_batch_ex.  Both sides evaluate the same
float32 fused-multiply-add chains in element order, so the bar is bit-exact equality of every output byte."""
import ctypes

import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

from helpers import GUARD, tiny_workload

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    from paper_2609_22441_b200 import binding, build

    build.build()
    binding.lib()
    return binding


def _member(wl, dim, n_chunks, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    m = (scale * rng.standard_normal((wl.batch.n_req, n_chunks * dim))).astype(np.float16)
    if wl.batch.n_req > 1:
        m[-1, :dim] = 0  # one request with an all-zero first medoid
    return m


def _want(wl, member, first, dim, n_chunks, first_degree_only=False):
    s, b = wl.store, wl.batch
    rows, mask = oracle.join_workload(wl, first_degree_only=first_degree_only, n_threads=4)
    cos = oracle.cosine_features(s.doc_feats, member, b.cand_idx, b.cand_offsets, first, dim, n_chunks)
    return np.concatenate([rows.reshape(len(mask), -1), cos], axis=1), mask


def _gpu(B, store, db, member_dev, flags, n_max=0):
    flags |= B.CCR_FLAG_COSINE
    out_b = store.out_row_bytes(flags)
    n = db.n_req * n_max if n_max else db.total_cands
    rows_buf = torch.full((GUARD + n * out_b + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    mask_buf = torch.full((GUARD + n + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    B.ccr_join_batch_ex(store, db.n_req, db.total_cands, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets,
                        db.cand_idx, db.cand_offsets, db.req_feats, rows_buf[GUARD:], mask_buf[GUARD:], flags, None, n_max,
                        member_dev)
    torch.cuda.synchronize()
    rb, mb = rows_buf.cpu().numpy(), mask_buf.cpu().numpy()
    assert (rb[:GUARD] == 0xA5).all() and (rb[GUARD + n * out_b:] == 0xA5).all(), "write outside out_rows"
    assert (mb[:GUARD] == 0xA5).all() and (mb[GUARD + n:] == 0xA5).all(), "write outside out_mask"
    return rb[GUARD:GUARD + n * out_b].reshape(n, out_b), mb[GUARD:GUARD + n]


def _check(B, wl, first, dim, n_chunks, flag_sets, seed=0, scale=1.0, tunings=((0, 0),), first_degree_only=False):
    member = _member(wl, dim, n_chunks, seed, scale)
    want_rows, want_mask = _want(wl, member, first, dim, n_chunks, first_degree_only)
    store = B.store_from_workload(wl)
    store.set_cosine(first, dim, n_chunks)
    db = B.DeviceBatch(wl.batch)
    mdev = torch.from_numpy(member).cuda()
    try:
        assert store.out_row_bytes(B.CCR_FLAG_COSINE) == store.out_row_bytes(0) + 32
        for tuning in tunings:
            if any(tuning):
                store.set_tuning(*tuning)
            for name, flags in flag_sets:
                if first_degree_only:
                    flags |= B.CCR_FLAG_FIRST_DEGREE_ONLY
                rows, mask = _gpu(B, store, db, mdev, flags)
                assert np.array_equal(mask, want_mask), (wl.name, name)
                if not np.array_equal(rows, want_rows):
                    bad = np.nonzero((rows != want_rows).any(axis=1))[0]
                    j = bad[0]
                    raise AssertionError("%s/%s: %d rows differ, first %d: got %s want %s" % (
                        wl.name, name, len(bad), j, rows[j, -32:].copy().view(np.float16), want_rows[j, -32:].copy().view(np.float16)))
        assert store.device_status() == B.CCR_OK
    finally:
        store.free()


def _paths(B):
    return [("ws", 0), ("ws+static", B.CCR_FLAG_STATIC_SPLIT), ("ws+global", B.CCR_FLAG_FORCE_GLOBAL),
            ("ws+sampled", B.CCR_FLAG_FORCE_SAMPLED)]


def _special_values(wl, first, dim, seed):
    """Zero item embeddings, infinities and NaNs, huge and tiny magnitudes in some rows."""
    d = wl.store.doc_feats
    rng = np.random.default_rng(seed)
    n = d.shape[0]
    pick = lambda k: rng.integers(0, n, size=max(1, n // k))
    d[pick(9), first:first + dim] = 0
    d[pick(11), first + int(rng.integers(0, dim))] = np.float16(np.inf)
    d[pick(13), first + int(rng.integers(0, dim))] = np.float16(np.nan)
    d[pick(7), first:first + dim] *= np.float16(200.0)
    d[pick(7), first:first + dim] *= np.float16(1e-3)
    return wl


@pytest.mark.parametrize("seed,dim,n_chunks,first", [(0, 50, 3, 8), (1, 50, 3, 0), (2, 64, 4, 0), (3, 7, 1, 56), (4, 1, 2, 32),
                                                      (5, 33, 4, 24), (6, 50, 3, 8), (7, 8, 3, 48)])
def test_tiny_batches_every_shape_of_the_embedding(B, seed, dim, n_chunks, first):
    rng = np.random.default_rng(40 + seed)
    second = bool(seed & 1)
    wl = tiny_workload(900 + seed, int(rng.integers(1, 80)), 20, int(rng.integers(1, 5)), 16, int(rng.integers(1, 120)),
                       second, 4 if seed % 3 == 0 else 0, doc_dim=64, doc_dtype=np.float16)
    _special_values(wl, first, dim, seed)
    _check(B, wl, first, dim, n_chunks, _paths(B), seed, tunings=((0, 0), (512, 0, 3, 2, 1)))
    if second:
        _check(B, wl, first, dim, n_chunks, [("ws", 0)], seed, first_degree_only=True)


@pytest.mark.parametrize("second", [False, True])
def test_scaled_config1_with_the_papers_embedding_shape(B, second):
    """Benchmark row widths (128 fp16 document features, of which 50 are the item embedding), 3 x 50 medoids."""
    wl = W.config1(n_docs=120_000, n_req=6, n_cand=7_000, second_degree=second)
    _special_values(wl, 8, 50, 1)
    _check(B, wl, 8, 50, 3, _paths(B), 3, tunings=((0, 0), (768, 0, 5, 8, 2)))
    _check(B, wl, 72, 50, 3, [("ws", 0)], 4, scale=25.0)


def test_padded_layout_with_cosine(B):
    wl = W.config1(n_docs=50_000, n_req=5, n_cand=3_000)
    s, b = wl.store, wl.batch
    member = _member(wl, 50, 3, 8)
    want_rows, want_mask = _want(wl, member, 8, 50, 3)
    store = B.store_from_workload(wl)
    store.set_cosine(8, 50, 3)
    db = B.DeviceBatch(b)
    try:
        n_max = 3_100
        rows, mask = _gpu(B, store, db, torch.from_numpy(member).cuda(), 0, n_max)
        out_b = rows.shape[1]
        T, M = rows.reshape(b.n_req, n_max, out_b), mask.reshape(b.n_req, n_max)
        for r in range(b.n_req):
            c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
            assert np.array_equal(T[r, :c1 - c0], want_rows[c0:c1]) and np.array_equal(M[r, :c1 - c0], want_mask[c0:c1])
            assert not T[r, c1 - c0:].any() and not M[r, c1 - c0:].any()
    finally:
        store.free()


def test_argument_errors(B):
    wl = tiny_workload(3, 30, 10, 2, 8, 20, False, 0, doc_dim=64, doc_dtype=np.float16)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    L = B.lib()
    member = torch.zeros((2, 150), dtype=torch.float16, device="cuda")
    rows = torch.empty((db.total_cands, store.out_row_bytes(B.CCR_FLAG_COSINE)), dtype=torch.uint8, device="cuda")
    mask = torch.empty((db.total_cands,), dtype=torch.uint8, device="cuda")

    def ex(flags, member_emb=member, struct_bytes=None):
        io = B.ccr_join_io(ctypes.sizeof(B.ccr_join_io) if struct_bytes is None else struct_bytes, db.n_req, db.total_cands,
                           db.max_edge_len, 0, db.edge_keys.data_ptr(), db.edge_feats.data_ptr(), db.edge_offsets.data_ptr(),
                           db.cand_idx.data_ptr(), db.cand_offsets.data_ptr(), None,
                           None if member_emb is None else member_emb.data_ptr(), rows.data_ptr(), mask.data_ptr())
        return L.ccr_join_batch_ex(store.handle, ctypes.byref(io), flags, None)

    try:
        assert ex(B.CCR_FLAG_COSINE) == B.CCR_ERR_INVALID_ARG                      # not configured yet
        spec = lambda *a: ctypes.byref(B.ccr_cosine_spec(*a))
        assert L.ccr_docstore_set_cosine(store.handle, spec(4, 50, 3, 0)) == B.CCR_ERR_INVALID_ARG   # item_first not a multiple of 8
        assert L.ccr_docstore_set_cosine(store.handle, spec(16, 50, 3, 0)) == B.CCR_ERR_INVALID_ARG  # runs past the 64-value row
        assert L.ccr_docstore_set_cosine(store.handle, spec(0, 65, 3, 0)) == B.CCR_ERR_UNSUPPORTED
        assert L.ccr_docstore_set_cosine(store.handle, spec(0, 50, 5, 0)) == B.CCR_ERR_UNSUPPORTED
        assert L.ccr_docstore_set_cosine(store.handle, spec(0, 0, 3, 0)) == B.CCR_ERR_INVALID_ARG
        assert L.ccr_docstore_set_cosine(store.handle, spec(8, 50, 3, 0)) == B.CCR_OK
        assert ex(B.CCR_FLAG_COSINE, member_emb=None) == B.CCR_ERR_INVALID_ARG
        assert ex(B.CCR_FLAG_COSINE | B.CCR_FLAG_TWO_PHASE) == B.CCR_ERR_UNSUPPORTED
        assert ex(B.CCR_FLAG_COSINE | B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE) == B.CCR_ERR_UNSUPPORTED
        assert ex(B.CCR_FLAG_COSINE, struct_bytes=8) == B.CCR_ERR_INVALID_ARG
        assert ex(B.CCR_FLAG_COSINE) == B.CCR_OK
        assert ex(0) == B.CCR_OK                                                    # same entry without the section
        with pytest.raises(B.CcrError):                                             # the plain entry has no member argument
            B.ccr_join_batch(store, db.n_req, db.total_cands, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets,
                             db.cand_idx, db.cand_offsets, None, rows, mask, B.CCR_FLAG_COSINE)
        assert L.ccr_docstore_set_cosine(store.handle, None) == B.CCR_OK
        assert ex(B.CCR_FLAG_COSINE) == B.CCR_ERR_INVALID_ARG
        torch.cuda.synchronize()
        f32 = tiny_workload(3, 30, 10, 2, 8, 20, False, 0)  # float32 document rows
        st32 = B.store_from_workload(f32)
        try:
            assert L.ccr_docstore_set_cosine(st32.handle, spec(0, 2, 1, 0)) == B.CCR_ERR_UNSUPPORTED
        finally:
            st32.free()
    finally:
        store.free()


def test_config1_full_size_with_cosine(B):
    """The benchmark's batch (64 x 30,000 candidates, 1M documents) with the paper's 3 x 50 embedding shape."""
    wl = W.config1()
    _check(B, wl, 8, 50, 3, [("ws", 0)], 12)
