"""GPU parity of ccr_resolve_ids (Eq. 6: document id -> position or -1) against the CPU oracle."""
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


def _queries(rng, ids, n):
    if len(ids) == 0:
        return rng.integers(-5, 50, size=n).astype(np.int64)
    present = ids[rng.integers(0, len(ids), size=n)]
    q = np.where(rng.random(n) < 0.8, present, present + 1)  # ids are even: +1 is never indexed
    q[:4] = [ids[0] - 2, ids[-1] + 2, -9, np.iinfo(np.int64).max]
    return q.astype(np.int64)


# sizes around every boundary of the search tree (windows of 8 keys, a top level of at most 2,048 keys)
@pytest.mark.parametrize("n_ids", [0, 1, 2, 7, 8, 9, 31, 32, 33, 1023, 1024, 1025, 2047, 2048, 2049, 2055, 2056, 16383, 16384,
                                   16385, 8 * 16384 - 1, 8 * 16384, 8 * 16384 + 5, 32 * 16384 + 5, 3_000_000])
@pytest.mark.parametrize("with_positions", [False, True])
def test_resolve_matches_oracle(B, n_ids, with_positions):
    rng = np.random.default_rng(n_ids + with_positions)
    ids = (np.cumsum(rng.integers(1, 6, size=n_ids)) * 2).astype(np.int64)
    pos = rng.permutation(n_ids).astype(np.int32) if with_positions else None
    q = _queries(rng, ids, 20_000)
    want = oracle.resolve_ids(ids, q, pos)
    ix = B.IdIndex(ids, pos)
    out = torch.full((len(q) + 64,), -7, dtype=torch.int32, device="cuda")
    ix.resolve(torch.from_numpy(q).cuda(), out[32:32 + len(q)])
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert (got[:32] == -7).all() and (got[32 + len(q):] == -7).all()
    assert np.array_equal(got[32:32 + len(q)], want)
    if n_ids:
        assert (want >= 0).mean() > 0.5
    ix.free()


@pytest.mark.parametrize("n_ids", [0, 1, 9, 2048, 2049, 16385, 8 * 16384 + 5, 3_000_000])
@pytest.mark.parametrize("n_q", [(1 << 20), (1 << 20) + 37])
def test_resolve_large_batches_take_the_lane_per_query_top_search(B, n_ids, n_q):
    """From 2^20 queries on the kernel searches the top level a lane per query and hands the queries to the lane
    groups by shuffles: same results, ragged last warp included, the largest int64 among the queries."""
    rng = np.random.default_rng(n_ids + n_q)
    ids = (np.cumsum(rng.integers(1, 6, size=n_ids)) * 2).astype(np.int64)
    pos = rng.permutation(n_ids).astype(np.int32) if n_ids % 2 else None
    q = _queries(rng, ids, n_q)
    want = oracle.resolve_ids(ids, q, pos)
    ix = B.IdIndex(ids, pos)
    out = torch.full((len(q) + 64,), -7, dtype=torch.int32, device="cuda")
    ix.resolve(torch.from_numpy(q).cuda(), out[32:32 + len(q)])
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert (got[:32] == -7).all() and (got[32 + len(q):] == -7).all()
    assert np.array_equal(got[32:32 + len(q)], want)
    ix.free()


@pytest.mark.parametrize("n_ids", [5, 8, 13, 2048, 2051, 40_001])
def test_resolve_with_the_largest_int64_as_an_id(B, n_ids):
    """Keys beyond the end of a level count as +infinity inside the kernel; an id equal to that value is still
    found when it is indexed and not found when it is not."""
    rng = np.random.default_rng(n_ids)
    top = np.iinfo(np.int64).max
    ids = (np.cumsum(rng.integers(1, 6, size=n_ids)) * 2).astype(np.int64)
    for with_top in (False, True):
        if with_top:
            ids[-1] = top
        q = np.concatenate([ids, ids + 1, [top, top - 1, -1, 0]]).astype(np.int64)  # ids + 1 wraps for the top id
        want = oracle.resolve_ids(ids, q)
        assert (want[-4] >= 0) == with_top
        ix = B.IdIndex(ids)
        out = torch.full((len(q),), -7, dtype=torch.int32, device="cuda")
        ix.resolve(torch.from_numpy(q).cuda(), out)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), want)
        ix.free()


def test_resolve_a_few_hundred_million_ids(B):
    """The paper's scale: a sorted array of a few hundred million ids resident in HBM."""
    if torch.cuda.mem_get_info()[0] < 12 * 2**30:
        pytest.skip("needs ~8 GB of free device memory")
    n = 300_000_000
    g = torch.Generator(device="cuda")
    g.manual_seed(W.config_seed(5))
    ids = torch.cumsum(torch.randint(1, 4, (n,), generator=g, device="cuda", dtype=torch.int64), 0) * 2
    ix = B.IdIndex(ids)  # device source
    host = ids.cpu().numpy()
    del ids
    rng = np.random.default_rng(3)
    q = _queries(rng, host, 8 * 30_000)
    got = ix.resolve(torch.from_numpy(q).cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.resolve_ids(host, q))
    ix.free()
    # device-side ids given from the host must resolve identically (smaller index)
    ix2 = B.IdIndex(host[:5_000_000])
    q2 = _queries(rng, host[:5_000_000], 30_000)
    assert np.array_equal(ix2.resolve(torch.from_numpy(q2).cuda()).cpu().numpy(), oracle.resolve_ids(host[:5_000_000], q2))
    ix2.free()


def test_resolved_positions_feed_the_join(B):
    """ids -> positions on the device -> join, against the oracle's join on the oracle's positions; unknown
    ids become -1 and give zero rows."""
    wl = W.config1(n_docs=60_000, n_req=5, n_cand=4_000)
    s, b = wl.store, wl.batch
    rng = np.random.default_rng(4)
    doc_ids = (np.cumsum(rng.integers(1, 5, size=s.n_docs)) * 2).astype(np.int64)  # id of the doc at rank i
    positions = rng.permutation(s.n_docs).astype(np.int32)                          # where that doc lives in the store
    inv = np.empty(s.n_docs, np.int64)
    inv[positions] = np.arange(s.n_docs)
    q = doc_ids[inv[b.cand_idx]]           # the ids a request would carry for these candidates
    q[::50] += 1                           # some unknown ids
    want_pos = oracle.resolve_ids(doc_ids, q, positions)
    assert (want_pos[::50] == -1).all() and np.array_equal(np.delete(want_pos, np.s_[::50]), np.delete(b.cand_idx, np.s_[::50]))
    ix = B.IdIndex(doc_ids, positions)
    got_pos = ix.resolve(torch.from_numpy(q).cuda())
    assert np.array_equal(got_pos.cpu().numpy(), want_pos)
    store = B.store_from_workload(wl)
    db = B.DeviceBatch(b)
    db.cand_idx = got_pos
    rows, mask = gpu_join(store, db)
    want = oracle.join_workload(W.Workload("r", 0, s, W.Batch(**{**b.__dict__, "cand_idx": want_pos})))
    assert np.array_equal(rows, want[0]) and np.array_equal(mask, want[1])
    assert not rows[::50].reshape(len(rows[::50]), -1)[:, :320].any()
    store.free()
    ix.free()
