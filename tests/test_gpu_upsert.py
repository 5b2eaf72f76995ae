"""GPU parity of the store write path (Section 6.2, ingestion step 3: scatter a batch to assigned positions).
The store has no read-back call, and what matters is what the join then computes, so the check is: join over the
upserted device store == oracle join over the oracle-upserted host store, byte for byte, with candidates that
name every row of the store."""
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


def _all_rows_batch(wl, extra_seed=0):
    """The workload's requests with candidate lists replaced by: every store position once (shuffled), plus the
    original candidates."""
    s, b = wl.store, wl.batch
    rng = np.random.default_rng(extra_seed)
    keys_l, feats_l, cands_l = [], [], []
    for r in range(b.n_req):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        keys_l.append(b.edge_keys[e0:e1])
        feats_l.append(b.edge_feats[e0:e1])
        cands_l.append(np.concatenate([rng.permutation(s.n_docs).astype(np.int32), b.cand_idx[c0:c1]]))
    return W.assemble_batch(keys_l, feats_l, cands_l, b.req_feats, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype)


def _host_state(s):
    return [s.doc_feats.copy(), s.author_ids.copy(), None if s.actor_ids is None else s.actor_ids.copy(),
            None if s.actor_types is None else s.actor_types.copy()]


def _apply(B, store, state, pos, doc=None, auth=None, act=None, typ=None, stream=None):
    """One batch on both sides: device store through the C ABI, host state through the oracle."""
    dev = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    store.upsert(dev(pos.astype(np.int32)), dev(doc), dev(auth), dev(act), dev(typ), stream=stream)
    state[:] = oracle.upsert(state[0], state[1], pos, doc, auth, state[2], state[3], act, typ)


def _compare(B, store, state, batch, s, flag_sets=(("ws", 0),)):
    want_rows, want_mask = oracle.join(state[0], state[1], batch.edge_keys, batch.edge_feats, batch.edge_offsets,
                                       batch.cand_idx, batch.cand_offsets, req_feats=batch.req_feats, actor_ids=state[2],
                                       actor_types=state[3], reduce_sum_mask=s.reduce_sum_mask, n_threads=4)
    db = B.DeviceBatch(batch)
    for name, flags in flag_sets:
        rows, mask = gpu_join(store, db, flags)
        assert np.array_equal(mask, want_mask), name
        assert np.array_equal(rows, want_rows), name
    assert store.device_status() == B.CCR_OK


@pytest.mark.parametrize("seed", range(8))
def test_tiny_stores_every_combination_of_sources(B, seed):
    second = bool(seed & 1)
    rng = np.random.default_rng(500 + seed)
    n_docs = int(rng.integers(1, 70))
    wl = tiny_workload(600 + seed, n_docs, 20, int(rng.integers(1, 4)), 16, 30, second, 4 if seed % 3 == 0 else 0)
    s = wl.store
    batch = _all_rows_batch(wl, seed)
    donor = W.make_store(np.random.default_rng(700 + seed), 7 * (n_docs + 4), 20, 4, np.float32, max_actors=4 if second else 0,
                         reduce_sum_mask=s.reduce_sum_mask)
    store = B.store_from_workload(wl)
    state = _host_state(s)
    kernels = [("auto", 0), ("ws", B.CCR_FLAG_WARP_SPECIALISED), ("2phase", B.CCR_FLAG_TWO_PHASE)]
    try:
        _compare(B, store, state, batch, s, kernels)  # before any write
        used = 0
        for what in ("all", "doc", "ids", "slots", "types", "all"):
            m = int(rng.integers(0, n_docs + 1))
            pos = rng.permutation(n_docs)[:m].astype(np.int64)
            # a few rows aimed outside the store write nothing
            junk = rng.choice(np.array([-1, -5, n_docs, n_docs + 3, 2**31 - 1]), size=int(rng.integers(0, 4)))
            pos = rng.permutation(np.concatenate([pos, junk]))
            d = slice(used, used + len(pos))
            used += len(pos)
            doc = donor.doc_feats[d] if what in ("all", "doc") else None
            auth = donor.author_ids[d] if what in ("all", "ids") else None
            act = donor.actor_ids[d] if second and what in ("all", "ids", "slots") else None
            typ = donor.actor_types[d] if second and what in ("all", "types") else None
            _apply(B, store, state, pos, doc, auth, act, typ)
            _compare(B, store, state, batch, s, kernels)
        L = B.lib()
        assert L.ccr_docstore_upsert(store.handle, -1, None, None, None, None, None, None) == B.CCR_ERR_INVALID_ARG
        assert L.ccr_docstore_upsert(store.handle, 0, None, None, None, None, None, None) == B.CCR_OK
        assert L.ccr_docstore_upsert(store.handle, 3, None, None, None, None, None, None) == B.CCR_ERR_INVALID_ARG
        if not second:
            p = torch.zeros(3, dtype=torch.int32, device="cuda")
            junk = torch.zeros(64, dtype=torch.int64, device="cuda")
            assert L.ccr_docstore_upsert(store.handle, 3, p.data_ptr(), None, None, junk.data_ptr(), None,
                                         None) == B.CCR_ERR_INVALID_ARG
    finally:
        store.free()


@pytest.mark.parametrize("second", [False, True])
def test_scaled_config1_batches_of_new_and_updated_documents(B, second):
    """200k-document store, benchmark row widths; three batches (new rows, updates of old rows, engager-slot
    updates only), then the benchmark-shaped join over old and new rows."""
    wl = W.config1(n_docs=200_000, n_req=6, n_cand=6_000, second_degree=second)
    s, b = wl.store, wl.batch
    donor = W.config1(seed=4242, n_docs=200_000, n_req=1, n_cand=10, second_degree=second).store
    rng = np.random.default_rng(17)
    store = B.store_from_workload(wl)
    state = _host_state(s)
    try:
        for m, what in ((60_000, "all"), (33_333, "all"), (20_001, "slots")):
            pos = rng.permutation(s.n_docs)[:m].astype(np.int64)
            src = rng.permutation(s.n_docs)[:m]
            if what == "slots" and not second:
                _apply(B, store, state, pos, auth=donor.author_ids[src])
            elif what == "slots":
                _apply(B, store, state, pos, act=donor.actor_ids[src], typ=donor.actor_types[src])
            else:
                _apply(B, store, state, pos, donor.doc_feats[src], donor.author_ids[src],
                       donor.actor_ids[src] if second else None, donor.actor_types[src] if second else None)
        _compare(B, store, state, b, s, [("auto", 0), ("ws", B.CCR_FLAG_WARP_SPECIALISED), ("2phase", B.CCR_FLAG_TWO_PHASE)])
    finally:
        store.free()


def test_join_on_one_stream_while_new_documents_arrive_on_another(B):
    """The paper's order (write the rows, then publish the ids): requests in flight only name old positions, new
    documents land on positions nobody can name yet.  Joins over the old rows run on one stream while batches
    of new rows are scattered on another; every join result equals the oracle on the old rows, and once the
    writes are done a join that names the new rows equals the oracle on the final store."""
    n_live, n_new = 150_000, 50_000
    wl = W.config1(n_docs=n_live + n_new, n_req=8, n_cand=8_000)
    s, b = wl.store, wl.batch
    old_only = b.cand_idx % n_live  # every in-flight request names live rows only
    b.cand_idx = old_only.astype(np.int32)
    donor = W.config1(seed=99, n_docs=n_new, n_req=1, n_cand=10).store
    store = B.store_from_workload(wl)
    state = _host_state(s)
    want_rows, want_mask = oracle.join(state[0], state[1], b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx,
                                       b.cand_offsets, req_feats=b.req_feats, n_threads=4)
    db = B.DeviceBatch(b)
    s_join, s_ing = torch.cuda.Stream(), torch.cuda.Stream()
    rng = np.random.default_rng(5)
    new_pos = (n_live + rng.permutation(n_new)).astype(np.int64)
    batches = np.array_split(np.arange(n_new), 10)
    dev_batches = [(torch.from_numpy(new_pos[i].astype(np.int32)).cuda(), torch.from_numpy(donor.doc_feats[i]).cuda(),
                    torch.from_numpy(donor.author_ids[i]).cuda()) for i in batches]
    outs = [(torch.empty((b.total_cands, store.out_row_bytes()), dtype=torch.uint8, device="cuda"),
             torch.empty((b.total_cands,), dtype=torch.uint8, device="cuda")) for _ in range(10)]
    torch.cuda.synchronize()
    try:
        for k in range(10):
            p, d, a = dev_batches[k]
            store.upsert(p, d, a, stream=s_ing)
            B.join_batch(store, db, 0, outs[k][0], outs[k][1], stream=s_join)
        torch.cuda.synchronize()
        for rows, mask in outs:
            assert np.array_equal(mask.cpu().numpy(), want_mask)
            assert np.array_equal(rows.cpu().numpy(), want_rows)
        for i in batches:
            state[:] = oracle.upsert(state[0], state[1], new_pos[i], donor.doc_feats[i], donor.author_ids[i])
        # now the ids are "published": requests may name the new rows
        b.cand_idx = rng.integers(0, n_live + n_new, size=b.total_cands).astype(np.int32)
        _compare(B, store, state, b, s)
    finally:
        store.free()
