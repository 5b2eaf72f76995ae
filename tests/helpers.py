"""Shared test helpers: tiny random problems and the GPU call with guard bytes around the outputs."""
import numpy as np

from paper_2609_22441_b200 import workloads as W

GUARD = 256


def tiny_workload(seed, n_docs, alphabet, n_req, kmax, nmax, second, req_dim, doc_dim=4, doc_dtype=np.float32,
                  edge_dim=8, sum_mask=0b10110100):
    """Tiny problem with ids from a tiny alphabet so that hits, misses, repeats, empty requests and
    unresolved / out-of-range positions are all common."""
    rng = np.random.default_rng(seed)
    store = W.make_store(rng, n_docs, alphabet, doc_dim, doc_dtype, max_actors=4 if second else 0,
                         reduce_sum_mask=sum_mask if second else 0)
    keys_l, feats_l, cands_l = [], [], []
    # negatives, ties, +-0, a subnormal, values whose sums overflow, infinities and two NaN encodings
    vals = np.concatenate([np.array([-2.0, -0.5, 0.0, 0.25, 0.5, 1.0, 1.5, 3.0, 1000.0, 6e-5, 60000.0, -0.0], np.float16),
                           np.array([0x7C00, 0xFC00, 0x7E00, 0x7C01], np.uint16).view(np.float16)])
    for _ in range(n_req):
        k = int(rng.integers(0, min(kmax, alphabet) + 1))
        keys, _ = W.make_viewer(rng, alphabet, k, edge_dim, np.float16)
        feats = rng.choice(vals, size=(k, edge_dim))
        n = int(rng.integers(0, nmax + 1))
        cands_l.append(rng.integers(-1, n_docs + 1, size=n).astype(np.int32))
        keys_l.append(keys)
        feats_l.append(feats)
    req = rng.standard_normal((n_req, req_dim)).astype(np.float32) if req_dim else None
    batch = W.assemble_batch(keys_l, feats_l, cands_l, req, edge_dim, np.float16, req_dim, np.float32)
    return W.Workload("tiny", seed, store, batch)


def gpu_join(store, db, flags=0):
    """Run ccr_join_batch into buffers framed by guard bytes; returns numpy (rows, mask) after checking
    that no byte outside the output ranges was written."""
    import torch

    from paper_2609_22441_b200 import binding as B

    out_b = store.out_row_bytes(flags)
    n = db.total_cands
    dev = torch.device("cuda", store.device)
    rows_buf = torch.full((GUARD + n * out_b + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
    mask_buf = torch.full((GUARD + n + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
    rows = rows_buf[GUARD:GUARD + n * out_b].view(n, out_b) if n else rows_buf[GUARD:GUARD].view(0, out_b)
    mask = mask_buf[GUARD:GUARD + n]
    B.ccr_join_batch(store, db.n_req, n, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets, db.cand_idx,
                     db.cand_offsets, db.req_feats, rows, mask, flags)
    torch.cuda.synchronize(dev)
    rb, mb = rows_buf.cpu().numpy(), mask_buf.cpu().numpy()
    assert (rb[:GUARD] == 0xA5).all() and (rb[GUARD + n * out_b:] == 0xA5).all(), "write outside out_rows"
    assert (mb[:GUARD] == 0xA5).all() and (mb[GUARD + n:] == 0xA5).all(), "write outside out_mask"
    return rb[GUARD:GUARD + n * out_b].reshape(n, out_b), mb[GUARD:GUARD + n]


def upload_generated_store(B, wl, device=0, keep_rows_of=None, keep_all=False):
    return B.store_from_generated(wl, device, keep_rows_of, keep_all)


def sampled_oracle_rows(wl, kept, J, first_degree_only):
    """Oracle rows and mask for the flat candidate indices J (ascending) of a workload whose doc features
    exist on the host only for the sampled docs: the sample is re-expressed as a compact problem (store =
    the sampled docs, candidates = 0..len(J)-1, same requests) and given to the unmodified oracle."""
    from oracle import oracle

    s, b = wl.store, wl.batch
    J = np.asarray(J, dtype=np.int64)
    docs = b.cand_idx[J].astype(np.int64)
    ok = (docs >= 0) & (docs < s.n_docs)
    where = np.searchsorted(kept["idx"], np.where(ok, docs, kept["idx"][0]))
    assert np.array_equal(kept["idx"][where][ok], docs[ok])
    feats = kept["rows"][where]
    cand = np.where(ok, np.arange(len(J)), -1).astype(np.int32)
    safe = np.where(ok, docs, 0)
    req_of = np.searchsorted(b.cand_offsets, J, side="right") - 1
    co = np.searchsorted(req_of, np.arange(b.n_req + 1), side="left").astype(np.int64)
    return oracle.join(
        feats, s.author_ids[safe], b.edge_keys, b.edge_feats, b.edge_offsets, cand, co, req_feats=b.req_feats,
        actor_ids=None if s.actor_ids is None else s.actor_ids[safe],
        actor_types=None if s.actor_types is None else s.actor_types[safe],
        reduce_sum_mask=s.reduce_sum_mask, first_degree_only=first_degree_only, n_threads=4)


def request_oracle_rows(wl, full, r, first_degree_only, cand_idx=None):
    """Oracle rows and mask of ALL candidates of request r of a production-scale workload whose feature matrix
    lives on the device only (`full`: the generator's output, i.e. an input, as a device tensor).  The rows of
    the request's docs are gathered from that input matrix to the host and the request is re-expressed as a
    compact single-request problem (store = those rows, candidates = 0..n-1) for the unmodified oracle."""
    import torch

    from oracle import oracle

    s, b = wl.store, wl.batch
    cand_idx = b.cand_idx if cand_idx is None else cand_idx
    c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
    e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
    docs = cand_idx[c0:c1].astype(np.int64)
    ok = (docs >= 0) & (docs < s.n_docs)
    safe = np.where(ok, docs, 0)
    feats = full.index_select(0, torch.from_numpy(safe).to(full.device)).cpu().numpy()
    n = c1 - c0
    return oracle.join(
        feats, s.author_ids[safe], b.edge_keys[e0:e1], b.edge_feats[e0:e1], np.array([0, e1 - e0], np.int64),
        np.where(ok, np.arange(n), -1).astype(np.int32), np.array([0, n], np.int64),
        req_feats=None if b.req_feats is None else b.req_feats[r:r + 1],
        actor_ids=None if s.actor_ids is None else s.actor_ids[safe],
        actor_types=None if s.actor_types is None else s.actor_types[safe],
        reduce_sum_mask=s.reduce_sum_mask, first_degree_only=first_degree_only, n_threads=4)
