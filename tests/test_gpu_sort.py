"""GPU parity of ccr_sort_edges (Algorithm 1 step 1) against the CPU oracle, and of the join fed with
device-sorted records."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

from helpers import gpu_join

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    from paper_2609_22441_b200 import binding, build

    build.build()
    return binding


def _shuffle_records(batch, seed, duplicate_keys=False):
    rng = np.random.default_rng(seed)
    keys, feats = batch.edge_keys.copy(), batch.edge_feats.copy()
    for r in range(batch.n_req):
        a, z = int(batch.edge_offsets[r]), int(batch.edge_offsets[r + 1])
        p = rng.permutation(z - a)
        keys[a:z], feats[a:z] = batch.edge_keys[a:z][p], batch.edge_feats[a:z][p]
        if duplicate_keys and z - a > 4:
            keys[a:z:3] = keys[a]  # many equal keys: the order among them must be the input order
    return keys, feats


def _gpu_sort(B, store, keys, feats, eo, with_perm=True):
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    k_in, f_in, o = dev(keys), dev(feats), dev(eo)
    guard = 64
    k_buf = torch.full((len(keys) + 2 * guard,), -7, dtype=torch.int64, device="cuda")
    f_buf = torch.full((feats.shape[0] + 2 * guard, feats.shape[1]), 7.0, dtype=torch.float16, device="cuda")
    p_buf = torch.full((len(keys) + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    E = len(keys)
    k_out, f_out, p_out = k_buf[guard:guard + E], f_buf[guard:guard + E], p_buf[guard:guard + E]
    n_req = len(eo) - 1
    max_len = int(np.max(np.diff(eo))) if n_req else 0
    B.ccr_sort_edges(store, n_req, max_len, k_in, f_in, o, k_out, f_out, p_out if with_perm else None)
    torch.cuda.synchronize()
    assert (k_buf[:guard] == -7).all() and (k_buf[guard + E:] == -7).all()
    assert (f_buf[:guard] == 7).all() and (f_buf[guard + E:] == 7).all()
    assert (p_buf[:guard] == -7).all() and (p_buf[guard + E:] == -7).all()
    return k_out, f_out, p_out


@pytest.mark.parametrize("dups", [False, True])
def test_sort_matches_oracle_on_config1_and_the_join_accepts_it(B, dups):
    wl = W.config1(n_docs=100_000, n_req=24, n_cand=3_000)
    b = wl.batch
    keys_u, feats_u = _shuffle_records(b, 1, duplicate_keys=dups)
    want_k, want_f, want_p = oracle.sort_edges(keys_u, feats_u, b.edge_offsets)
    store = B.store_from_workload(wl)
    k, f, p = _gpu_sort(B, store, keys_u, feats_u, b.edge_offsets)
    assert np.array_equal(k.cpu().numpy(), want_k)
    assert np.array_equal(p.cpu().numpy(), want_p)
    assert np.array_equal(f.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
    if not dups:
        # sorted on the device, joined on the device == oracle join of the originally sorted records
        db = B.DeviceBatch(b)
        db.edge_keys, db.edge_feats = k.contiguous(), f.contiguous()
        rows, mask = gpu_join(store, db)
        want_rows, want_mask = oracle.join_workload(wl)
        assert np.array_equal(rows, want_rows) and np.array_equal(mask, want_mask)
    store.free()


@pytest.mark.parametrize("lens", [[0, 1, 2, 3, 31, 32, 33, 1023, 1024, 1025, 4097], [18_999, 19_000, 7], [19_001, 40_000, 5, 0, 65_537],
                                  [4096, 100, 0, 4095, 129, 128, 127]])  # the last: no list beyond one chunk, one block per list
def test_sort_lengths_around_the_block_and_shared_memory_limits(B, lens):
    rng = np.random.default_rng(sum(lens))
    keys = np.concatenate([rng.integers(0, 10 * max(n, 1), size=n) for n in lens] + [np.empty(0, np.int64)]).astype(np.int64)
    feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
    eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    want_k, want_f, want_p = oracle.sort_edges(keys, feats, eo)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)  # a store with 128-byte edge rows
    store = B.store_from_workload(wl)
    k, f, p = _gpu_sort(B, store, keys, feats, eo)
    assert np.array_equal(k.cpu().numpy(), want_k) and np.array_equal(p.cpu().numpy(), want_p)
    assert np.array_equal(f.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
    if max(lens) <= 19_000:
        k2, f2, _ = _gpu_sort(B, store, keys, feats, eo, with_perm=False)
        assert np.array_equal(k2.cpu().numpy(), want_k) and np.array_equal(f2.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
    else:
        with pytest.raises(B.CcrError) as e:
            _gpu_sort(B, store, keys, feats, eo, with_perm=False)
        assert e.value.status == B.CCR_ERR_INVALID_ARG
    store.free()


def test_sort_with_keys_that_cannot_share_a_word_with_the_index(B):
    """Keys near INT64_MAX (and negative ones, outside the join's contract but legal for the sort) force the
    two-array network; mixed with small-key requests in one launch."""
    rng = np.random.default_rng(9)
    imax = np.iinfo(np.int64).max
    lens = [700, 5000, 64, 3000]
    parts = [imax - rng.integers(0, 10_000, size=lens[0]), rng.integers(0, 1 << 40, size=lens[1]),
             rng.integers(-50, 50, size=lens[2]), rng.integers(0, 1 << 62, size=lens[3])]
    keys = np.concatenate(parts).astype(np.int64)
    feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
    eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    want_k, want_f, want_p = oracle.sort_edges(keys, feats, eo)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
    store = B.store_from_workload(wl)
    k, f, p = _gpu_sort(B, store, keys, feats, eo)
    assert np.array_equal(k.cpu().numpy(), want_k) and np.array_equal(p.cpu().numpy(), want_p)
    assert np.array_equal(f.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
    store.free()


@pytest.mark.parametrize("case", ["few_long", "many_long", "mixed_unpackable", "powers_of_two", "very_long"])
def test_sort_chunked_path(B, case):
    """With perm_out, lists are sorted in chunks of 4,096 records by one block each and the chunks merged pairwise,
    one launch per doubling of the run length (a list of K records takes ceil(log2(K / 4096)) merges and its words
    end in the key array or in the scratch area accordingly) — unless a list's keys cannot share a word with the
    index; those stay on the one-block path inside the same launch sequence."""
    rng = np.random.default_rng({"few_long": 1, "many_long": 2, "mixed_unpackable": 3, "powers_of_two": 4, "very_long": 5}[case])
    imax = np.iinfo(np.int64).max
    if case == "few_long":
        lens = [4097, 9000, 20_000, 3, 0, 12_288, 4096, 16_385]
        keyf = [lambda n: rng.integers(0, 50 * max(n, 1), size=n)] * len(lens)
    elif case == "many_long":
        lens = [5000] * 70 + [100, 8191]
        keyf = [lambda n: rng.integers(0, 1 << 30, size=n)] * len(lens)
    elif case == "mixed_unpackable":
        lens = [6000, 10_000, 5000, 7000, 50]
        keyf = [lambda n: rng.integers(0, 1 << 40, size=n), lambda n: imax - rng.integers(0, 1 << 20, size=n),
                lambda n: rng.integers(-1000, 1000, size=n), lambda n: rng.integers(0, 1000, size=n),  # many ties
                lambda n: rng.integers(0, 1 << 40, size=n)]
    elif case == "powers_of_two":
        lens = [8192, 16_384, 32_768, 8193, 16_383]
        keyf = [lambda n: rng.integers(0, 1 << 45, size=n)] * len(lens)
    else:  # four, five and six merges; few distinct keys in the longest (ties across every run boundary)
        lens = [131_073, 70_000, 12_289, 65_536]
        keyf = [lambda n: rng.integers(0, 97, size=n), lambda n: rng.integers(0, 1 << 44, size=n),
                lambda n: rng.integers(0, 1 << 20, size=n), lambda n: np.arange(n)[::-1].copy()]
    keys = np.concatenate([f(n) for f, n in zip(keyf, lens)] + [np.empty(0, np.int64)]).astype(np.int64)
    feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
    eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    want_k, want_f, want_p = oracle.sort_edges(keys, feats, eo)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
    store = B.store_from_workload(wl)
    try:
        for _ in range(2):  # twice: the flag left in the output rows by the first call must not confuse the second
            k, f, p = _gpu_sort(B, store, keys, feats, eo)
            assert np.array_equal(k.cpu().numpy(), want_k) and np.array_equal(p.cpu().numpy(), want_p)
            assert np.array_equal(f.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
    finally:
        store.free()


def test_sort_with_an_untruthful_length_bound_stays_in_bounds(B):
    """max_edge_len below the longest list (a broken promise): lists are cut at the bound — their first
    max_edge_len records sorted among themselves, nothing written behind, no access outside the arrays."""
    rng = np.random.default_rng(12)
    lens = [9000, 300, 12_000]
    keys = np.concatenate([rng.integers(0, 1 << 30, size=n) for n in lens]).astype(np.int64)
    feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
    eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
    store = B.store_from_workload(wl)
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    try:
        for bound in (5000, 200):
            k_out = torch.full((len(keys),), -7, dtype=torch.int64, device="cuda")
            f_out = torch.full(feats.shape, 7.0, dtype=torch.float16, device="cuda")
            p_out = torch.full((len(keys),), -7, dtype=torch.int32, device="cuda")
            B.ccr_sort_edges(store, len(lens), bound, dev(keys), dev(feats), dev(eo), k_out, f_out, p_out)
            torch.cuda.synchronize()
            k, f, p = k_out.cpu().numpy(), f_out.cpu().numpy(), p_out.cpu().numpy()
            for r, n in enumerate(lens):
                a, m = int(eo[r]), min(n, bound)
                order = np.argsort(keys[a:a + m], kind="stable")
                assert np.array_equal(k[a:a + m], keys[a:a + m][order]) and np.array_equal(p[a:a + m], order)
                assert np.array_equal(f[a:a + m].view(np.uint16), feats[a:a + m][order].view(np.uint16))
                assert (k[a + m:a + n] == -7).all() and (p[a + m:a + n] == -7).all() and (f[a + m:a + n] == 7).all()
    finally:
        store.free()


def test_sort_a_list_with_more_row_tiles_than_a_grid_has_rows(B):
    """16.8M records of 128-byte rows: the row gather needs more than 65,535 tiles for the list, so its grid (and
    only its grid) takes the folded one-dimensional form; a short list rides along.  Keys and permutation are
    compared in full, the rows on 200,000 sampled records and the short list."""
    if torch.cuda.mem_get_info()[0] < 12 * 2**30:
        pytest.skip("needs ~6 GB of free device memory")
    rng = np.random.default_rng(77)
    lens = [16_800_000, 5000]
    E = sum(lens)
    keys = rng.integers(0, 1 << 34, size=E, dtype=np.int64)
    eo = np.array([0, lens[0], E], dtype=np.int64)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
    store = B.store_from_workload(wl)
    try:
        k_in = torch.from_numpy(keys).cuda()
        # rows made on the device: row i = 16 int32 lanes of (i * 2654435761 + lane) — 128 bytes like the store's edge rows
        i = torch.arange(E, dtype=torch.int64, device="cuda").unsqueeze(1)
        f_in = ((i * 2654435761 + torch.arange(32, dtype=torch.int64, device="cuda")) & 0x7fffffff).to(torch.int32)
        assert f_in.shape[1] * 4 == wl.batch.edge_row_bytes
        k_out, f_out = torch.empty_like(k_in), torch.empty_like(f_in)
        p_out = torch.empty(E, dtype=torch.int32, device="cuda")
        B.ccr_sort_edges(store, 2, lens[0], k_in, f_in, torch.from_numpy(eo).cuda(), k_out, f_out, p_out)
        torch.cuda.synchronize()
        k, p = k_out.cpu().numpy(), p_out.cpu().numpy()
        want_k, _, want_p = oracle.sort_edges(keys, np.zeros((E, 1), np.uint8), eo)  # one-byte rows: keys and order only
        assert np.array_equal(k, want_k) and np.array_equal(p, want_p)
        sample = np.concatenate([rng.integers(0, lens[0], size=200_000), np.arange(lens[0], E),
                                 np.array([0, 1, lens[0] - 1])]).astype(np.int64)
        src = np.where(sample < lens[0], p[sample], lens[0] + p[sample])
        got = f_out[torch.from_numpy(sample).cuda()].cpu().numpy()
        want = f_in[torch.from_numpy(src).cuda()].cpu().numpy()
        assert np.array_equal(got, want)
    finally:
        store.free()


@pytest.mark.parametrize("seed", range(12))
def test_sort_random_batches(B, seed):
    """Random batches: list lengths drawn around every boundary of the chunked path (empty, a few records, one
    chunk, one record more, two / four / eight chunks +- 1, tens of thousands), key ranges from a handful of
    distinct values (ties across every run boundary) to 2^44, with and without the permutation output."""
    rng = np.random.default_rng(1000 + seed)
    n_req = int(rng.integers(1, 40))
    with_perm = bool(seed % 3 != 2)
    pools = [lambda: 0, lambda: int(rng.integers(1, 50)), lambda: int(rng.integers(1000, 6000)),
             lambda: int(rng.integers(4090, 4103)), lambda: int(rng.integers(8185, 8200)),
             lambda: int(rng.integers(16380, 16390)), lambda: int(rng.integers(10_000, 19_000)),
             lambda: int(rng.integers(32_760, 32_775)) if with_perm else int(rng.integers(18_000, 19_000))]
    lens = [pools[int(rng.integers(0, len(pools)))]() for _ in range(n_req)]
    hi = [3, 100, 1 << 20, 1 << 44][int(rng.integers(0, 4))]
    keys = rng.integers(0, hi, size=sum(lens), dtype=np.int64)
    feats = rng.standard_normal((len(keys), 64)).astype(np.float16)
    eo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    want_k, want_f, want_p = oracle.sort_edges(keys, feats, eo)
    wl = W.config3(n_docs=1000, n_req=1, n_cand=10, gen_doc_feats=True, extra_pools=0)
    store = B.store_from_workload(wl)
    try:
        k, f, p = _gpu_sort(B, store, keys, feats, eo, with_perm=with_perm)
        assert np.array_equal(k.cpu().numpy(), want_k)
        assert np.array_equal(f.cpu().numpy().view(np.uint16), want_f.view(np.uint16))
        if with_perm:
            assert np.array_equal(p.cpu().numpy(), want_p)
    finally:
        store.free()
