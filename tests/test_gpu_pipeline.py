"""The steps around the join chained on the device, as a serving request flows through them: ingestion scatter of
new documents (Section 6.2) -> document ids to positions (Eq. 6) -> compaction of the resolved candidates and
padded layout (Section 6.3.1) -> per-request sort of the unsorted affinity records (Algorithm 1 step 1) -> the
join with the derived cosine section (Algorithm 1 steps 2-4, Section 4.1.2).  No host round trip between the
steps; the result is compared byte for byte with the same chain of oracle functions."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    from paper_2609_22441_b200 import binding, build

    build.build()
    binding.lib()
    return binding


@pytest.mark.parametrize("second", [False, True])
def test_request_flow_end_to_end(B, second):
    rng = np.random.default_rng(31 + second)
    wl = W.config1(n_docs=80_000, n_req=12, n_cand=5_000, second_degree=second, edge_lo=20, edge_hi=6_000)
    s, b = wl.store, wl.batch
    n_live = 70_000  # positions >= n_live are free slots for new documents
    # document ids: position p holds id doc_id[p]; the id index is sorted by id
    doc_id = rng.permutation(10 * s.n_docs)[:s.n_docs].astype(np.int64)
    # a request names candidates by id; some ids are unknown, some belong to documents that arrive in this test
    cand_pos = b.cand_idx.astype(np.int64)
    cand_ids = doc_id[cand_pos]
    unknown = rng.random(len(cand_ids)) < 0.03
    cand_ids = np.where(unknown, -5 - np.arange(len(cand_ids)), cand_ids)
    # affinity records arrive unsorted
    keys_in, feats_in = b.edge_keys.copy(), b.edge_feats.copy()
    for r in range(b.n_req):
        a, z = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        p = rng.permutation(z - a)
        keys_in[a:z], feats_in[a:z] = b.edge_keys[a:z][p], b.edge_feats[a:z][p]
    member = rng.standard_normal((b.n_req, 150)).astype(np.float16)
    # ingestion: the documents at positions >= n_live are "new": the device store starts without them
    new_pos = np.arange(n_live, s.n_docs, dtype=np.int64)
    rng.shuffle(new_pos)

    # ---------------- oracle chain
    order = np.argsort(doc_id, kind="stable")
    want_pos = oracle.resolve_ids(doc_id[order], cand_ids, order.astype(np.int32))
    o_keys, o_feats, _ = oracle.sort_edges(keys_in, feats_in, b.edge_offsets)
    kw = dict(req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types, reduce_sum_mask=s.reduce_sum_mask)
    n_max = int(np.diff(b.cand_offsets).max())
    want_T, want_M, n_valid, src = oracle.join_padded(s.doc_feats, s.author_ids, o_keys, o_feats, b.edge_offsets, want_pos,
                                                      b.cand_offsets, n_max=n_max, **kw)
    want_cos = oracle.cosine_features(s.doc_feats, member, want_pos, b.cand_offsets, 8, 50, 3)[src]

    # ---------------- device chain
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    store = B.Docstore(s.n_docs, s.doc_dim, s.doc_dtype, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype, s.max_actors,
                       s.reduce_sum_mask, 0)
    ix = None
    try:
        store.upload(0, s.doc_feats[:n_live], s.author_ids[:n_live], None if not second else s.actor_ids[:n_live],
                     None if not second else s.actor_types[:n_live])
        store.set_cosine(8, 50, 3)
        ix = B.IdIndex(dev(doc_id[order]), dev(order.astype(np.int32)))
        store.upsert(dev(new_pos.astype(np.int32)), dev(s.doc_feats[new_pos]), dev(s.author_ids[new_pos]),
                     dev(s.actor_ids[new_pos]) if second else None, dev(s.actor_types[new_pos]) if second else None)
        pos = ix.resolve(dev(cand_ids))
        C, n_req = len(cand_ids), b.n_req
        co = dev(b.cand_offsets)
        idx = torch.empty(C, dtype=torch.int32, device="cuda")
        offs = torch.empty(n_req + 1, dtype=torch.int64, device="cuda")
        src_d = torch.empty(C, dtype=torch.int32, device="cuda")
        B.ccr_compact_valid(store, n_req, C, pos, co, idx, offs, src_d)
        k_in, f_in, eo = dev(keys_in), dev(feats_in), dev(b.edge_offsets)
        k_out, f_out = torch.empty_like(k_in), torch.empty_like(f_in)
        perm = torch.empty(len(keys_in), dtype=torch.int32, device="cuda")
        B.ccr_sort_edges(store, n_req, b.max_edge_len, k_in, f_in, eo, k_out, f_out, perm)
        flags = B.CCR_FLAG_COSINE
        out_b = store.out_row_bytes(flags)
        T = torch.empty((n_req, n_max, out_b), dtype=torch.uint8, device="cuda")
        M = torch.empty((n_req, n_max), dtype=torch.uint8, device="cuda")
        B.ccr_join_batch_ex(store, n_req, C, b.max_edge_len, k_out, f_out, eo, idx, offs, dev(b.req_feats), T, M, flags, None,
                            n_max, dev(member))
        torch.cuda.synchronize()
        assert store.device_status() == B.CCR_OK
        assert np.array_equal(pos.cpu().numpy(), want_pos)
        assert np.array_equal(np.diff(offs.cpu().numpy()), n_valid)
        V = int(n_valid.sum())
        assert np.array_equal(src_d[:V].cpu().numpy(), src)
        assert np.array_equal(k_out.cpu().numpy(), o_keys)
        got_T, got_M = T.cpu().numpy(), M.cpu().numpy()
        assert np.array_equal(got_M, want_M)
        k = 0
        for r in range(n_req):
            n_r = int(n_valid[r])
            assert np.array_equal(got_T[r, :n_r, :out_b - 32], want_T[r, :n_r]), r
            assert np.array_equal(got_T[r, :n_r, out_b - 32:], want_cos[k:k + n_r]), r
            assert not got_T[r, n_r:].any(), r
            k += n_r
        assert (want_M & 1).sum() > 0.3 * V and unknown.sum() > 0 and (want_pos >= n_live).sum() > 0
    finally:
        if ix is not None:
            ix.free()
        store.free()
