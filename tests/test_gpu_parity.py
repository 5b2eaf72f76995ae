"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, byte for byte.

The join is indexing and copying (plus a fixed-order fp16 reduction for second-degree stores whose
rounding both sides take in fp32 with one final round-to-nearest-even), so the bar is bit-exact equality
of every output row and mask byte."""
import ctypes

import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

from helpers import gpu_join, tiny_workload

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    from paper_2609_22441_b200 import binding, build

    build.build()
    binding.lib()
    return binding


def _variants(B, include_smem=True):
    """Every key-search path, each through the warp-specialised kernel (default: dynamic chunks; and with the
    static split) and the two-phase kernel."""
    v = [("auto", 0), ("global", B.CCR_FLAG_FORCE_GLOBAL), ("sampled", B.CCR_FLAG_FORCE_SAMPLED)]
    if include_smem:
        v.append(("smem", B.CCR_FLAG_FORCE_SMEM))
    # without a kernel flag a small launch takes the two-phase kernel and a large one the warp-specialised kernel
    v.append(("global+warp-search", B.CCR_FLAG_FORCE_GLOBAL | B.CCR_FLAG_WARP_SEARCH))
    return (v + [(n + "+2phase", f | B.CCR_FLAG_TWO_PHASE) for n, f in v] +
            [(n + "+ws", f | B.CCR_FLAG_WARP_SPECIALISED) for n, f in v] +
            [(n + "+static", f | B.CCR_FLAG_STATIC_SPLIT) for n, f in v])


def _check(B, wl, flag_sets, first_degree_only=False, tunings=((0, 0),)):
    want_rows, want_mask = oracle.join_workload(wl, first_degree_only=first_degree_only, n_threads=4)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    try:
        for tuning in tunings:
            tile, cap = tuning[0], tuning[1]
            if any(tuning):
                store.set_tuning(*tuning)
            for name, flags in flag_sets:
                if first_degree_only:
                    flags |= B.CCR_FLAG_FIRST_DEGREE_ONLY
                rows, mask = gpu_join(store, db, flags)
                assert np.array_equal(mask, want_mask), (wl.name, name, tile, cap)
                assert rows.shape == want_rows.shape
                if not np.array_equal(rows, want_rows):
                    bad = np.nonzero((rows != want_rows).any(axis=1))[0]
                    raise AssertionError("%s/%s tile=%d cap=%d: %d rows differ, first %d" %
                                         (wl.name, name, tile, cap, len(bad), bad[0]))
        assert store.device_status() == B.CCR_OK
    finally:
        store.free()
    return want_rows, want_mask


# ------------------------------------------------------------------ the benchmark configurations
def test_config0_single_tiny_request_all_search_paths(B):
    wl = W.config0()
    _check(B, wl, _variants(B))
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])


def test_config1_batched_first_degree_full_size(B):
    wl = W.config1()
    assert wl.batch.total_cands == 64 * 30_000 and wl.out_row_bytes() == 384
    _check(B, wl, _variants(B), tunings=((0, 0), (512, 0, 1, 1, 1), (2048, 0, 14, 2, 3), (768, 0, 5, 8, 2), (256, 0, 3, 1, 0)))
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])


def test_config2a_second_degree_on_config0_shape(B):
    wl = W.config0(second_degree=True)
    assert wl.out_row_bytes() == 384
    _, mask = _check(B, wl, _variants(B))
    assert (mask >> 1).any() and (mask >> 5).any()
    _check(B, wl, [("auto", 0)], first_degree_only=True)
    ws = W.sort_candidates_by_author(wl)
    _check(B, ws, [("sorted-second", B.CCR_FLAG_CANDS_SORTED)])
    _check(B, ws, [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)], first_degree_only=True)


def test_config2b_second_degree_on_config1_shape_full_size(B):
    wl = W.config1(second_degree=True)
    assert wl.out_row_bytes() == 448
    # large sub-tiles and other warp splits: the engager work lists address candidates by their index in the sub-tile
    _check(B, wl, [("auto", 0), ("global", B.CCR_FLAG_FORCE_GLOBAL), ("ws", B.CCR_FLAG_WARP_SPECIALISED)],
           tunings=((0, 0), (4096, 0, 12, 4, 0), (2048, 0, 8, 8, 0), (768, 0, 14, 1, 0)))


def test_config3_scaled_store_long_edge_lists(B):
    # production shape at 1/25 of the store: K log-uniform up to 20000 (longer than the default staging
    # budget, so the sampled top-of-tree path runs), 128-byte edge rows, second-degree store joined
    # first-degree-only as in the headline run, then fully
    wl = W.config3(n_docs=2_000_000, n_req=12, n_cand=20_000, gen_doc_feats=True, extra_pools=0)
    assert wl.batch.max_edge_len > 4096
    _check(B, wl, _variants(B), first_degree_only=True, tunings=((0, 0), (512, 1000), (2048, 20_000), (256, 7)))
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)], first_degree_only=True,
           tunings=((0, 0), (256, 64)))
    _check(B, wl, [("auto", 0)])


def test_more_requests_than_the_kernel_mirrors_in_shared_memory(B):
    """Batches of up to 1024 requests keep their offsets in shared memory; larger ones read them from global
    memory.  1500 small requests, first and second degree, every kernel."""
    for second in (False, True):
        wl = W.config1(n_docs=30_000, n_req=1500, n_cand=150, second_degree=second, edge_lo=3, edge_hi=80)
        assert wl.batch.n_req == 1500
        _check(B, wl, [("auto", 0), ("ws", B.CCR_FLAG_WARP_SPECIALISED), ("static", B.CCR_FLAG_STATIC_SPLIT),
                       ("2phase", B.CCR_FLAG_TWO_PHASE), ("global+ws", B.CCR_FLAG_FORCE_GLOBAL | B.CCR_FLAG_WARP_SPECIALISED)])


# ------------------------------------------------------------------ ragged / degenerate inputs
@pytest.mark.parametrize("seed", range(12))
def test_tiny_random_batches(B, seed):
    second = bool(seed % 2)
    wl = tiny_workload(seed, n_docs=37 + seed, alphabet=20 + 3 * seed, n_req=1 + seed, kmax=16, nmax=70,
                       second=second, req_dim=4 * (seed % 3 == 0))
    _check(B, wl, _variants(B), tunings=((256, 0), (0, 0)))
    if second:
        _check(B, wl, [("auto", 0)], first_degree_only=True)
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)], first_degree_only=second,
           tunings=((256, 3),))


def test_generic_widths_take_the_runtime_variant(B):
    # 96-byte doc rows, 16-byte edge rows, 16 bytes of request features: none of the compiled-in layouts
    wl = tiny_workload(99, n_docs=500, alphabet=300, n_req=7, kmax=120, nmax=900, second=False, req_dim=4,
                       doc_dim=24, edge_dim=8)
    _check(B, wl, _variants(B))
    wl2 = tiny_workload(98, n_docs=500, alphabet=300, n_req=7, kmax=120, nmax=900, second=True, req_dim=0,
                        doc_dim=24, edge_dim=8)
    _check(B, wl2, _variants(B))


def _manual(keys_l, cand_l, author_ids, n_docs=None, edge_dim=32, doc_dim=64, seed=0):
    rng = np.random.default_rng(seed)
    n_docs = n_docs or len(author_ids)
    store = W.Store(n_docs=n_docs, doc_dim=doc_dim, doc_dtype=np.dtype(np.float32),
                    author_ids=np.asarray(author_ids, np.int64),
                    doc_feats=rng.standard_normal((n_docs, doc_dim)).astype(np.float32))
    feats_l = [rng.random((len(k), edge_dim), dtype=np.float32).astype(np.float16) for k in keys_l]
    batch = W.assemble_batch([np.asarray(k, np.int64) for k in keys_l], feats_l,
                             [np.asarray(c, np.int32) for c in cand_l], None, edge_dim, np.float16, 0, np.float32)
    return W.Workload("manual", seed, store, batch)


def test_search_boundaries_and_empty_requests(B):
    imax = np.iinfo(np.int64).max
    authors = [0, 5, 7, 9, imax, imax - 1, -3, 6, 7, 7]
    keys = [[0, 7, imax], [], [7], [0, 7, imax], [5, 6, 9, imax - 1]]
    cands = [[0, 1, 2, 3, 4, 5, 6, 7, 2, 2, -1, 10], [1, 2, 3], [2, 8, 9, 0], [], [1, 7, 3, 5, 4, 2]]
    wl = _manual(keys, cands, authors)
    rows, mask = _check(B, wl, _variants(B), tunings=((256, 0), (0, 0)))
    assert list(mask[:12]) == [1, 0, 1, 0, 1, 0, 0, 0, 1, 1, 0, 0]
    assert list(mask[12:15]) == [0, 0, 0] and list(mask[15:19]) == [1, 1, 1, 0] and list(mask[19:]) == [1, 1, 1, 1, 0, 0]


def test_all_found_none_found_and_duplicates(B):
    rng = np.random.default_rng(3)
    authors = rng.integers(0, 1000, size=4000)
    all_keys = np.unique(authors)
    none_keys = np.arange(2000, 2600)
    cand = rng.integers(0, 4000, size=5000)  # with repeats
    wl = _manual([all_keys, none_keys, all_keys[::2]], [cand, cand, cand[:1]], authors)
    rows, mask = _check(B, wl, _variants(B))
    assert mask[:5000].all() and not mask[5000:10000].any()


@pytest.mark.parametrize("k", [1, 2, 3, 255, 256, 257, 4095, 4096, 4097, 8191, 20_000, 65_536, 100_000])
def test_edge_list_lengths_around_every_path_threshold(B, k):
    # two requests so that the second one's keys start at an odd (8-byte aligned only) offset when k is odd
    rng = np.random.default_rng(k)
    n_docs = 30_000
    authors = rng.integers(0, 4 * k + 10, size=n_docs)
    keys1 = W.sorted_unique_sample(rng, 4 * k + 10, k)
    keys2 = W.sorted_unique_sample(rng, 4 * k + 10, k)
    cand = [rng.integers(0, n_docs, size=3000), rng.integers(0, n_docs, size=2500)]
    wl = _manual([keys1, keys2], cand, authors, edge_dim=8)
    fits_smem = k <= 20_000
    _check(B, wl, _variants(B, include_smem=fits_smem))
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])
    if not fits_smem:
        store = B.store_from_workload(wl)
        db = B.DeviceBatch(wl.batch)
        with pytest.raises(B.CcrError) as e:
            gpu_join(store, db, B.CCR_FLAG_FORCE_SMEM)
        assert e.value.status == B.CCR_ERR_UNSUPPORTED
        store.free()


@pytest.mark.parametrize("key_dist", ["clustered", "pareto"])
@pytest.mark.parametrize("k", [37, 4096, 13_000, 20_000])
def test_clustered_and_heavy_tailed_keys_through_every_search_path(B, key_dist, k):
    """Ids that a linear map of the key range cannot spread: a block of consecutive ids plus one id near the top
    of the int64 range (the whole block shares one bucket of such a map), and heavy-tailed gaps (dense runs
    separated by huge jumps).  Candidates hit the block's first and last keys, the far key, ids just outside
    the block and inside the gaps; two requests, so the second key list starts at an odd offset when k is odd."""
    rng = np.random.default_rng(1000 + k)
    n_docs = 40_000
    keys1 = W.make_keys(rng, 5_000_000, k, key_dist)
    keys2 = W.make_keys(rng, 5_000_000, k - 1, key_dist)
    near = np.concatenate([keys1, keys1 + 1, keys1 - 1, keys2, keys2[-1:] + 1, keys1[:1] - 1])
    authors = np.where(rng.random(n_docs) < 0.8, near[rng.integers(0, len(near), size=n_docs)],
                       rng.integers(0, 5_000_000, size=n_docs)).astype(np.int64)
    authors[:4] = [keys1[0], keys1[-1], keys1[-2], max(int(keys1[0]) - 1, 0)]
    cand = [np.concatenate([np.arange(4), rng.integers(0, n_docs, size=6000)]), rng.integers(0, n_docs, size=3500)]
    wl = _manual([keys1, keys2], cand, authors, edge_dim=32)
    _, mask = _check(B, wl, _variants(B), tunings=((0, 0), (256, 1000)))
    assert list(mask[:3]) == [1, 1, 1] and 0.1 < mask.mean() < 0.95
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])


@pytest.mark.parametrize("key_dist", ["clustered", "pareto"])
def test_batched_shape_with_non_uniform_keys_first_and_second_degree(B, key_dist):
    for second in (False, True):
        wl = W.config1(n_docs=200_000, n_req=16, n_cand=12_000, second_degree=second, key_dist=key_dist)
        _, mask = _check(B, wl, [("auto", 0), ("2phase", B.CCR_FLAG_TWO_PHASE), ("sampled", B.CCR_FLAG_FORCE_SAMPLED),
                                 ("global", B.CCR_FLAG_FORCE_GLOBAL)])
        assert 0.2 < (mask & 1).mean() < 0.7


def test_sorted_candidates_with_unresolved_positions_inside(B):
    """CCR_FLAG_CANDS_SORTED binds the resolved candidates only: -1 and out-of-range positions sit at the start,
    in the middle and at the end of sorted requests, alone and in runs, at sub-tile boundaries too."""
    wl = W.sort_candidates_by_author(W.config1(n_docs=60_000, n_req=5, n_cand=7_000))
    b = wl.batch
    rng = np.random.default_rng(11)
    cand = b.cand_idx.copy()
    for r in range(b.n_req):
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        holes = np.concatenate([rng.integers(c0, c1, size=40), [c0, c1 - 1, c0 + 1023, c0 + 1024, c0 + 2047],
                                np.arange(c0 + 3000, c0 + 3040)])
        cand[holes] = np.where(rng.random(len(holes)) < 0.5, -1, wl.store.n_docs + 5)
    cand[int(b.cand_offsets[3]):int(b.cand_offsets[3]) + 1500] = -1  # a whole sub-tile without a single author
    wl2 = W.Workload("sorted+holes", 0, wl.store, W.Batch(**{**b.__dict__, "cand_idx": cand}))
    _check(B, wl2, [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED),
                    ("merge+global", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE | B.CCR_FLAG_FORCE_GLOBAL),
                    ("merge+validate", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE | B.CCR_FLAG_VALIDATE)],
           tunings=((0, 0), (256, 64)))


def test_many_small_requests_in_one_launch(B):
    # hundreds of requests of 0..40 candidates: most blocks serve many request segments
    wl = tiny_workload(7, n_docs=3000, alphabet=900, n_req=700, kmax=300, nmax=40, second=False, req_dim=4,
                       doc_dim=64, edge_dim=32)
    _check(B, wl, _variants(B))
    _check(B, W.sort_candidates_by_author(wl), [("merge", B.CCR_FLAG_CANDS_SORTED | B.CCR_FLAG_TWO_PHASE), ("ws+sorted", B.CCR_FLAG_CANDS_SORTED)])


def test_batch_equals_single_request_launches(B):
    wl = W.config1(n_docs=50_000, n_req=6, n_cand=1500)
    s, b = wl.store, wl.batch
    store = B.store_from_workload(wl)
    rows, mask = gpu_join(store, B.DeviceBatch(b))
    for r in range(b.n_req):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        one = W.assemble_batch([b.edge_keys[e0:e1]], [b.edge_feats[e0:e1]], [b.cand_idx[c0:c1]],
                               b.req_feats[r:r + 1], b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype)
        r1, m1 = gpu_join(store, B.DeviceBatch(one))
        assert np.array_equal(r1, rows[c0:c1]) and np.array_equal(m1, mask[c0:c1])
    store.free()


# ------------------------------------------------------------------ host-buffer entry, validation, errors
def test_host_buffer_entry_matches_device_entry(B):
    wl = W.config1(n_docs=80_000, n_req=9, n_cand=4000)
    b = wl.batch
    want_rows, want_mask = oracle.join_workload(wl)
    store = B.store_from_workload(wl)
    ws = B.Workspace(store, b.n_req, b.total_cands, len(b.edge_keys))
    out_rows = torch.empty((b.total_cands, store.out_row_bytes()), dtype=torch.uint8).pin_memory()
    out_mask = torch.empty((b.total_cands,), dtype=torch.uint8).pin_memory()
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    args = [pin(b.edge_keys), pin(b.edge_feats.view(np.uint8)), pin(b.edge_offsets), pin(b.cand_idx),
            pin(b.cand_offsets), pin(b.req_feats.view(np.uint8))]
    for _ in range(2):
        out_rows.fill_(7)
        B.ccr_join_batch_host(store, ws, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *args,
                              out_rows, out_mask)
        torch.cuda.synchronize()
        assert np.array_equal(out_rows.numpy(), want_rows) and np.array_equal(out_mask.numpy(), want_mask)
    # the serving case: no host buffer for the rows, they stay in the workspace on the device; only the mask returns
    out_mask.fill_(9)
    B.ccr_join_batch_host(store, ws, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *args, None, out_mask)
    torch.cuda.synchronize()
    rows_ptr, mask_ptr = ws.outputs()
    class _View:  # the workspace's device buffer seen as a tensor (CUDA array interface)
        __cuda_array_interface__ = {"shape": (b.total_cands * store.out_row_bytes(),), "typestr": "|u1",
                                    "data": (rows_ptr, False), "version": 2}
    dev_rows = torch.as_tensor(_View(), device="cuda").view(b.total_cands, store.out_row_bytes())
    assert np.array_equal(dev_rows.cpu().numpy(), want_rows) and np.array_equal(out_mask.numpy(), want_mask)
    with pytest.raises(B.CcrError) as e:
        B.ccr_join_batch_host(store, ws, b.n_req, b.total_cands + 1, b.max_edge_len, len(b.edge_keys), *args,
                              out_rows, out_mask)
    assert e.value.status == B.CCR_ERR_INVALID_ARG
    ws.free()
    store.free()


def test_host_buffer_entry_pipelines_a_large_batch_in_request_groups(B):
    """Batches of several large requests cross PCIe in groups of requests while earlier groups are joined: very
    unequal requests (one of them empty, one holding a third of the candidates), twice in a row on one workspace,
    rows left on the device and rows copied back."""
    base = W.config1(n_docs=400_000, n_req=24, n_cand=60_000)
    b0 = base.batch
    rng = np.random.default_rng(3)
    sizes = rng.integers(5_000, 60_001, size=b0.n_req)
    sizes[5] = 0
    sizes[17] = 60_000
    keys_l, feats_l, cands_l = [], [], []
    for r in range(b0.n_req):
        e0, e1 = int(b0.edge_offsets[r]), int(b0.edge_offsets[r + 1])
        c0 = int(b0.cand_offsets[r])
        keys_l.append(b0.edge_keys[e0:e1])
        feats_l.append(b0.edge_feats[e0:e1])
        cands_l.append(b0.cand_idx[c0:c0 + int(sizes[r])])
    # one request of a third of all candidates (repeats are fine)
    cands_l[2] = np.concatenate([b0.cand_idx[int(b0.cand_offsets[2]):int(b0.cand_offsets[3])]] * 8)
    wl = W.Workload("ragged-large", 0, base.store, W.assemble_batch(keys_l, feats_l, cands_l, b0.req_feats, b0.edge_dim,
                                                                   b0.edge_dtype, b0.req_dim, b0.req_dtype))
    b = wl.batch
    assert b.total_cands > 1_100_000
    want_rows, want_mask = oracle.join_workload(wl, n_threads=4)
    store = B.store_from_workload(wl)
    ws = B.Workspace(store, b.n_req, b.total_cands, len(b.edge_keys))
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    args = [pin(b.edge_keys), pin(b.edge_feats.view(np.uint8)), pin(b.edge_offsets), pin(b.cand_idx),
            pin(b.cand_offsets), pin(b.req_feats.view(np.uint8))]
    out_b = store.out_row_bytes()
    out_mask = torch.empty((b.total_cands,), dtype=torch.uint8).pin_memory()
    rows_ptr, _ = ws.outputs()

    class _View:  # the workspace's device buffer seen as a tensor (CUDA array interface)
        __cuda_array_interface__ = {"shape": (b.total_cands * out_b,), "typestr": "|u1", "data": (rows_ptr, False), "version": 2}

    dev_rows = torch.as_tensor(_View(), device="cuda").view(b.total_cands, out_b)
    for _ in range(2):
        out_mask.fill_(9)
        dev_rows.fill_(7)
        torch.cuda.synchronize()
        B.ccr_join_batch_host(store, ws, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *args, None, out_mask)
        torch.cuda.synchronize()
        assert np.array_equal(out_mask.numpy(), want_mask)
        assert np.array_equal(dev_rows.cpu().numpy(), want_rows)
    out_rows = torch.empty((b.total_cands, out_b), dtype=torch.uint8).pin_memory()
    out_mask.fill_(9)
    B.ccr_join_batch_host(store, ws, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *args, out_rows, out_mask)
    torch.cuda.synchronize()
    assert np.array_equal(out_rows.numpy(), want_rows) and np.array_equal(out_mask.numpy(), want_mask)
    assert store.device_status() == B.CCR_OK
    ws.free()
    store.free()


def test_validate_flag_reports_broken_preconditions(B):
    wl = W.config1(n_docs=20_000, n_req=4, n_cand=500)
    store = B.store_from_workload(wl)
    good = B.DeviceBatch(wl.batch)
    gpu_join(store, good, B.CCR_FLAG_VALIDATE)

    def expect_validation(batch, flags=0):
        with pytest.raises(B.CcrError) as e:
            gpu_join(store, B.DeviceBatch(batch), B.CCR_FLAG_VALIDATE | flags)
        assert e.value.status == B.CCR_ERR_VALIDATION

    b = wl.batch
    keys = b.edge_keys.copy()
    e0 = int(b.edge_offsets[2])
    keys[e0], keys[e0 + 1] = keys[e0 + 1], keys[e0]  # one inversion inside request 2
    expect_validation(W.Batch(**{**b.__dict__, "edge_keys": keys}))
    keys = b.edge_keys.copy()
    keys[e0 + 1] = keys[e0]  # duplicate key
    expect_validation(W.Batch(**{**b.__dict__, "edge_keys": keys}))
    co = b.cand_offsets.copy()
    co[2], co[3] = co[3], co[2]  # non-monotone candidate offsets
    expect_validation(W.Batch(**{**b.__dict__, "cand_offsets": co}))
    # CANDS_SORTED on unsorted candidates is caught; on sorted ones it passes
    expect_validation(b, B.CCR_FLAG_CANDS_SORTED)
    gpu_join(store, B.DeviceBatch(W.sort_candidates_by_author(wl).batch), B.CCR_FLAG_VALIDATE | B.CCR_FLAG_CANDS_SORTED)
    # the store stays usable after a rejected call
    rows, mask = gpu_join(store, good)
    want_rows, want_mask = oracle.join_workload(wl)
    assert np.array_equal(rows, want_rows) and np.array_equal(mask, want_mask)
    store.free()


def test_unsorted_keys_and_false_sorted_promise_stay_in_bounds(B):
    # values are unspecified here; the guard bytes and a clean device status are what is checked
    wl = W.config1(n_docs=20_000, n_req=4, n_cand=3000)
    b = wl.batch
    rng = np.random.default_rng(0)
    keys = b.edge_keys.copy()
    rng.shuffle(keys)
    store = B.store_from_workload(wl)
    bad = B.DeviceBatch(W.Batch(**{**b.__dict__, "edge_keys": keys}))
    for _, flags in _variants(B):
        gpu_join(store, bad, flags)
    gpu_join(store, B.DeviceBatch(b), B.CCR_FLAG_CANDS_SORTED)  # candidates are not sorted
    gpu_join(store, bad, B.CCR_FLAG_CANDS_SORTED)
    assert store.device_status() == B.CCR_OK
    store.free()


def test_argument_errors_on_a_live_store(B):
    wl = W.config0(n_docs=5000, n_cand=1000, k=50)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(wl.batch)
    L = B.lib()
    out_rows = torch.empty((db.total_cands, 320), dtype=torch.uint8, device="cuda")
    out_mask = torch.empty((db.total_cands,), dtype=torch.uint8, device="cuda")

    def call(**kw):
        a = dict(n_req=db.n_req, total=db.total_cands, maxk=db.max_edge_len, keys=db.edge_keys.data_ptr(),
                 feats=db.edge_feats.data_ptr(), eo=db.edge_offsets.data_ptr(), ci=db.cand_idx.data_ptr(),
                 co=db.cand_offsets.data_ptr(), rows=out_rows.data_ptr(), mask=out_mask.data_ptr(), flags=0)
        a.update(kw)
        return L.ccr_join_batch(store.handle, a["n_req"], a["total"], a["maxk"], a["keys"], a["feats"], a["eo"], a["ci"],
                                a["co"], None, a["rows"], a["mask"], a["flags"], None)

    assert call() == B.CCR_OK
    assert call(n_req=-1) == B.CCR_ERR_INVALID_ARG
    assert call(total=-5) == B.CCR_ERR_INVALID_ARG
    assert call(rows=None) == B.CCR_ERR_INVALID_ARG
    assert call(rows=out_rows.data_ptr() + 8) == B.CCR_ERR_INVALID_ARG  # misaligned
    assert call(keys=db.edge_keys.data_ptr() + 8) == B.CCR_ERR_INVALID_ARG
    assert call(flags=B.CCR_FLAG_FORCE_SMEM | B.CCR_FLAG_FORCE_GLOBAL) == B.CCR_ERR_INVALID_ARG
    assert call(total=0) == B.CCR_OK and call(n_req=0, total=0) == B.CCR_OK
    assert store.out_row_bytes() == 320
    torch.cuda.synchronize()
    h = ctypes.c_void_p(store.handle.value)
    store.free()
    assert L.ccr_docstore_free(h) == B.CCR_ERR_BAD_HANDLE  # double free


def test_store_larger_than_device_memory_is_refused_before_any_allocation(B):
    free0 = torch.cuda.mem_get_info()[0]
    with pytest.raises(B.CcrError) as e:
        B.Docstore(2_000_000_000, 128, np.float16, 32)  # 512 GB of rows
    assert e.value.status == B.CCR_ERR_OOM
    with pytest.raises(B.CcrError) as e:
        B.Docstore(1_500_000_000, 128, np.float16, 32, max_actors=4)
    assert e.value.status == B.CCR_ERR_OOM
    assert abs(torch.cuda.mem_get_info()[0] - free0) < (64 << 20)  # nothing was allocated and kept


def test_joins_from_two_host_threads_on_one_store(B):
    """The launch counter is atomic and hands every launch its own scheduling words: two host threads join
    against one store at the same time, each on its own stream and into its own buffers."""
    import threading

    wl = W.config1(n_docs=200_000, n_req=16, n_cand=20_000)
    b = wl.batch
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(b)
    want_rows, want_mask = oracle.join_workload(wl, n_threads=4)
    n_calls = 40
    outs = [[(torch.full((b.total_cands, 384), 0x11, dtype=torch.uint8, device="cuda"),
              torch.full((b.total_cands,), 0x11, dtype=torch.uint8, device="cuda")) for _ in range(3)] for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    before = store.launch_count()
    errors = []

    def worker(t):
        try:
            for i in range(n_calls):
                rows, mask = outs[t][i % 3]
                B.ccr_join_batch(store, db.n_req, b.total_cands, db.max_edge_len, db.edge_keys, db.edge_feats,
                                 db.edge_offsets, db.cand_idx, db.cand_offsets, db.req_feats, rows, mask, 0, streams[t])
        except Exception as exc:  # pragma: no cover
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    torch.cuda.synchronize()
    assert not errors
    assert store.launch_count() == before + 2 * n_calls  # no increment was lost
    for t in range(2):
        for rows, mask in outs[t]:
            assert np.array_equal(mask.cpu().numpy(), want_mask) and np.array_equal(rows.cpu().numpy(), want_rows)
    assert store.device_status() == B.CCR_OK
    store.free()


def test_expired_device_wait_is_reported_and_the_store_stays_usable(B):
    """Failure reporting without a fault: a wait that nothing completes runs out of polls, the kernel returns,
    the status call reports it once, and the next join is bit-exact."""
    wl = W.config1(n_docs=30_000, n_req=3, n_cand=2_000)
    store = B.store_from_workload(wl)
    assert store.device_status() == B.CCR_OK
    store.selftest_wait()
    assert store.device_status() == B.CCR_ERR_DEVICE_WAIT
    assert store.device_status() == B.CCR_OK  # reading clears the word
    rows, mask = gpu_join(store, B.DeviceBatch(wl.batch))
    want_rows, want_mask = oracle.join_workload(wl)
    assert np.array_equal(rows, want_rows) and np.array_equal(mask, want_mask)
    assert store.device_status() == B.CCR_OK
    store.free()


def test_joins_in_flight_on_several_streams(B):
    """Launches of one store on different streams draw their chunks from different scheduling words."""
    wl = W.config1(n_docs=200_000, n_req=16, n_cand=20_000)
    b = wl.batch
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(b)
    want_rows, want_mask = oracle.join_workload(wl, n_threads=4)
    streams = [torch.cuda.Stream() for _ in range(4)]
    outs = [(torch.full((b.total_cands, 384), 0x11, dtype=torch.uint8, device="cuda"),
             torch.full((b.total_cands,), 0x11, dtype=torch.uint8, device="cuda")) for _ in range(12)]
    torch.cuda.synchronize()  # the fills ran on the default stream: finish them before other streams write
    for i, (rows, mask) in enumerate(outs):
        st = streams[i % len(streams)]
        B.ccr_join_batch(store, db.n_req, b.total_cands, db.max_edge_len, db.edge_keys, db.edge_feats,
                         db.edge_offsets, db.cand_idx, db.cand_offsets, db.req_feats, rows, mask, 0, st)
    torch.cuda.synchronize()
    for rows, mask in outs:
        assert np.array_equal(mask.cpu().numpy(), want_mask) and np.array_equal(rows.cpu().numpy(), want_rows)
    assert store.device_status() == B.CCR_OK
    store.free()


def test_back_to_back_joins_overlap_without_breaking_stream_order(B):
    """Consecutive joins on one stream move in behind each other (programmatic dependent launch).  What stream order
    promises must still hold: two different batches joined alternately into the SAME output buffers leave the last
    batch's rows (nothing of an earlier launch lands after a later one's); a kernel that rewrites the candidate
    positions between two joins is seen by the second join; and the result equals CCR_FLAG_NO_OVERLAP's."""
    wl_a = W.config1(n_docs=300_000, n_req=16, n_cand=30_000)
    rng = np.random.default_rng(9)
    b = wl_a.batch
    cand_b = b.cand_idx.copy()
    rng.shuffle(cand_b)
    wl_b = W.Workload("b", 0, wl_a.store, W.Batch(**{**b.__dict__, "cand_idx": cand_b}))
    want_a = oracle.join_workload(wl_a, n_threads=4)
    want_b = oracle.join_workload(wl_b, n_threads=4)
    store = B.store_from_workload(wl_a)
    da, db = B.DeviceBatch(wl_a.batch), B.DeviceBatch(wl_b.batch)
    rows = torch.empty((b.total_cands, 384), dtype=torch.uint8, device="cuda")
    mask = torch.empty((b.total_cands,), dtype=torch.uint8, device="cuda")

    def call(d, flags=0):
        B.ccr_join_batch(store, d.n_req, d.total_cands, d.max_edge_len, d.edge_keys, d.edge_feats, d.edge_offsets, d.cand_idx,
                         d.cand_offsets, d.req_feats, rows, mask, flags)

    for flags in (0, B.CCR_FLAG_NO_OVERLAP):
        for i in range(41):  # a, b, a, ... a
            call(da if i % 2 == 0 else db, flags)
        torch.cuda.synchronize()
        assert np.array_equal(mask.cpu().numpy(), want_a[1]) and np.array_equal(rows.cpu().numpy(), want_a[0])
        call(db, flags)
        torch.cuda.synchronize()
        assert np.array_equal(mask.cpu().numpy(), want_b[1]) and np.array_equal(rows.cpu().numpy(), want_b[0])
    # a torch kernel between two joins rewrites the second join's input: ordinary stream order applies to it
    scratch = da.cand_idx.clone()
    dc = B.DeviceBatch(wl_a.batch)
    dc.cand_idx = scratch
    for _ in range(10):
        call(da)
        scratch.copy_(db.cand_idx)   # now holds batch b's positions
        call(dc)
        torch.cuda.synchronize()
        assert np.array_equal(rows.cpu().numpy(), want_b[0])
        scratch.copy_(da.cand_idx)
    assert store.device_status() == B.CCR_OK
    store.free()


def test_upload_in_pieces_from_device_memory(B):
    wl = W.config0(n_docs=10_000, n_cand=3000, k=200, second_degree=True)
    s = wl.store
    store = B.Docstore(s.n_docs, s.doc_dim, s.doc_dtype, 32, np.float16, 0, np.float32, s.max_actors, s.reduce_sum_mask)
    for a in range(0, s.n_docs, 3333):
        z = min(s.n_docs, a + 3333)
        dev = lambda x: torch.from_numpy(np.ascontiguousarray(x[a:z])).cuda()
        store.upload(a, dev(s.doc_feats), dev(s.author_ids), dev(s.actor_ids), dev(s.actor_types))
    torch.cuda.synchronize()
    before = store.launch_count()  # uploads of a second-degree store launch their own (packing) kernels
    rows, mask = gpu_join(store, B.DeviceBatch(wl.batch))
    want_rows, want_mask = oracle.join_workload(wl)
    assert np.array_equal(rows, want_rows) and np.array_equal(mask, want_mask)
    assert store.launch_count() == before + 1
    # a partial upload (only the types of a few docs) leaves the other ids of those docs untouched
    types2 = s.actor_types.copy()
    types2[100:200] = (types2[100:200] + 1) % 3
    store.upload(100, None, None, None, np.ascontiguousarray(types2[100:200]))
    torch.cuda.synchronize()
    s2 = W.Store(**{**s.__dict__, "actor_types": types2})
    rows2, mask2 = gpu_join(store, B.DeviceBatch(wl.batch))
    want2 = oracle.join_workload(W.Workload("t", 0, s2, wl.batch))
    assert np.array_equal(rows2, want2[0]) and np.array_equal(mask2, want2[1])
    store.free()
