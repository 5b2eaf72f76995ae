"""ccr_join_payload_static — the join for callers that are not allowed to allocate device memory.

Such callers (a request handler inside a server that has already given all device memory to its own pool, or
one that cannot afford the device-wide stall of cudaMalloc / cudaFree) hand the request payload over in host
memory; the library copies it into a fixed 16 MiB device block that is part of its image and launches the
same kernel as ccr_join_batch.  The checks: rows and masks byte-identical to the CPU oracle and to
ccr_join_batch (the existing entry, device inputs) on two different batches called back to back — the second is
smaller, so stale bytes of the first would show —, no change of the device's free memory across the calls, the
refusal of a payload that does not fit the block, the refusal of scalars that disagree with the host offsets,
and that a device-side status raised while the entry is in use is still reported through the store.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_22441_b200 import workloads as W

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _pinned(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()


def test_static_payload_entry_matches_join_batch_twice_in_a_row():
    from paper_2609_22441_b200 import binding as B
    from paper_2609_22441_b200 import build

    build.build()
    first = W.config1(n_docs=120_000, n_req=12, n_cand=9_000)
    # a second, smaller batch against the same store: other requests, other sizes, an empty request inside
    rng = np.random.default_rng(5)
    b1 = first.batch
    keep = [0, 3, 4, 9]
    keys_l, feats_l, cands_l = [], [], []
    for r in keep:
        e0, e1 = int(b1.edge_offsets[r]), int(b1.edge_offsets[r + 1])
        c0, c1 = int(b1.cand_offsets[r]), int(b1.cand_offsets[r + 1])
        keys_l.append(b1.edge_keys[e0:e1])
        feats_l.append(b1.edge_feats[e0:e1])
        cands_l.append(rng.permutation(b1.cand_idx[c0:c1])[: 1000 + 777 * r])
    cands_l[2] = cands_l[2][:0]
    second = W.Workload("second", 0, first.store, W.assemble_batch(
        keys_l, feats_l, cands_l, b1.req_feats[keep], b1.edge_dim, b1.edge_dtype, b1.req_dim, b1.req_dtype))

    store = B.store_from_workload(first)
    assert B.lib().ccr_static_payload_capacity() == (16 << 20) - 256
    try:
        # first use on the device: looks up the block's address (and makes sure the library image is loaded)
        hb = first.batch
        warm = [_pinned(hb.edge_keys), _pinned(hb.edge_feats.view(np.uint8)), _pinned(hb.edge_offsets),
                _pinned(hb.cand_idx), _pinned(hb.cand_offsets), _pinned(hb.req_feats.view(np.uint8))]
        r0 = torch.empty((hb.total_cands, store.out_row_bytes()), dtype=torch.uint8, device="cuda")
        m0 = torch.empty((hb.total_cands,), dtype=torch.uint8, device="cuda")
        B.ccr_join_payload_static(store, hb.n_req, hb.total_cands, hb.max_edge_len, len(hb.edge_keys), *warm, r0, m0)
        torch.cuda.synchronize()
        for wl in (first, second):
            b = wl.batch
            oracle_rows, oracle_mask = oracle.join_workload(wl, n_threads=4)
            want_rows, want_mask = B.join_batch(store, B.DeviceBatch(b))
            torch.cuda.synchronize()
            rows = torch.full_like(want_rows, 0x5A)
            mask = torch.full_like(want_mask, 0x5A)
            host = [_pinned(b.edge_keys), _pinned(b.edge_feats.view(np.uint8)), _pinned(b.edge_offsets),
                    _pinned(b.cand_idx), _pinned(b.cand_offsets), _pinned(b.req_feats.view(np.uint8))]
            torch.cuda.synchronize()
            before = store.launch_count()
            free_before = torch.cuda.mem_get_info()[0]
            B.ccr_join_payload_static(store, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *host, rows, mask)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before  # the call took no device memory
            assert store.launch_count() == before + 1
            assert np.array_equal(mask.cpu().numpy(), oracle_mask)
            assert np.array_equal(rows.cpu().numpy(), oracle_rows)
            assert torch.equal(mask, want_mask)
            assert torch.equal(rows, want_rows)
        # a payload that cannot fit the fixed block is refused before anything is enqueued
        big_co = _pinned(np.array([0, 5_000_000], np.int64))
        one_eo = _pinned(np.array([0, 10], np.int64))
        with pytest.raises(B.CcrError) as e:
            B.ccr_join_payload_static(store, 1, 5_000_000, 10, 10, host[0], host[1], one_eo, host[3], big_co, host[5],
                                      rows, mask)
        assert e.value.status == B.CCR_ERR_UNSUPPORTED
        # scalars that disagree with the (host-readable) offsets are refused as well
        with pytest.raises(B.CcrError) as e:
            B.ccr_join_payload_static(store, b.n_req, b.total_cands - 1, b.max_edge_len, len(b.edge_keys), *host, rows, mask)
        assert e.value.status == B.CCR_ERR_INVALID_ARG
        with pytest.raises(B.CcrError) as e:
            B.ccr_join_payload_static(store, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys) - 1, *host, rows, mask)
        assert e.value.status == B.CCR_ERR_INVALID_ARG
        assert store.device_status() == B.CCR_OK
        # the entry keeps the store's own status word: a wait that ran out (here: the self-test's) is still
        # reported after a static call, not cleared by it
        store.selftest_wait()
        B.ccr_join_payload_static(store, b.n_req, b.total_cands, b.max_edge_len, len(b.edge_keys), *host, rows, mask)
        assert store.device_status() == B.CCR_ERR_DEVICE_WAIT
        assert store.device_status() == B.CCR_OK
        assert torch.equal(rows, want_rows) and torch.equal(mask, want_mask)
    finally:
        store.free()
