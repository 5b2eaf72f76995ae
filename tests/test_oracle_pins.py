"""Pins for the CPU oracle: checks against things other than itself.

  * the naive O(N*K) scan of Section 3.1 (pure Python, tiny inputs, hypothesis-generated);
  * Algorithm 1 steps 2-4 restated literally with library ops (torch.searchsorted / index_select / where);
  * the worked batching example of Section 6.3.1 (tests/golden/batching_example.txt);
  * set-intersection and concatenation invariants; boundary cases of Algorithm 1 step 3;
  * the oracle's fp16 <-> fp32 conversions against numpy's float16, exhaustively;
  * second-degree reduction special cases (the paper prints nothing for it).
"""
import os

import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import brute_force, oracle
from paper_2609_22441_b200 import workloads as W

from helpers import tiny_workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- fp16 conversions
def test_half_to_float_exhaustive_against_numpy():
    h = np.arange(65536, dtype=np.uint16)
    ref = h.view(np.float16).astype(np.float32)
    ref_bits = ref.view(np.uint32)
    got = np.array([oracle.half_to_float_bits(int(x)) for x in h], dtype=np.uint32)
    nan = np.isnan(ref)
    assert np.array_equal(got[~nan], ref_bits[~nan])
    assert np.all(np.isnan(got[nan].view(np.float32)))
    # round trip is the identity on every non-NaN half
    back = np.array([oracle.float_bits_to_half(int(b)) for b in got[~nan]], dtype=np.uint16)
    assert np.array_equal(back, h[~nan])


def test_float_to_half_rne_against_numpy():
    rng = np.random.default_rng(5)
    bits = [rng.integers(0, 2**32, size=120_000, dtype=np.uint64).astype(np.uint32)]
    # every tie between adjacent halves, and its two float neighbours (normal and subnormal range)
    h = np.arange(0, 0x7C00, dtype=np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    hi[-1] = 65536.0  # the "next half" after 65504 for rounding purposes
    mid = ((lo + hi) / 2).astype(np.float32)
    mb = mid.view(np.uint32)
    bits += [mb, mb + 1, mb - 1, mb | 0x80000000]
    # around the subnormal floor and the overflow threshold
    for v in (2.0**-25, 2.0**-24, 2.0**-26, 65504.0, 65519.99, 65520.0, 65536.0, 1e30, 1e-30, 0.0):
        f = np.array([v, -v], dtype=np.float32).view(np.uint32)
        bits += [f, f + 1, f - 1]
    bits = np.concatenate(bits).astype(np.uint32)
    f = bits.view(np.float32)
    keep = ~np.isnan(f)
    with np.errstate(over="ignore"):
        ref = f[keep].astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_bits_to_half(int(b)) for b in bits[keep]], dtype=np.uint16)
    assert np.array_equal(got, ref)
    assert oracle.float_bits_to_half(0x7FC00000) == 0x7FFF  # NaN is stored canonically


# ---------------------------------------------------------------- helpers
def _oracle(wl, **kw):
    return oracle.join_workload(wl, **kw)


def _brute(wl, **kw):
    s, b = wl.store, wl.batch
    return brute_force.join(
        s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets,
        req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types,
        reduce_sum_mask=s.reduce_sum_mask, **kw)


def _tiny(seed, n_docs, alphabet, n_req, kmax, nmax, second, req_dim):
    return tiny_workload(seed, n_docs, alphabet, n_req, kmax, nmax, second, req_dim)


# ---------------------------------------------------------------- brute force (naive scan) == oracle
@settings(max_examples=60, deadline=None, suppress_health_check=list(HealthCheck))
@given(seed=st.integers(0, 2**31), n_docs=st.integers(1, 40), alphabet=st.integers(1, 24),
       n_req=st.integers(0, 4), second=st.booleans(), req_dim=st.sampled_from([0, 4]))
def test_oracle_equals_naive_scan(seed, n_docs, alphabet, n_req, second, req_dim):
    wl = _tiny(seed, n_docs, alphabet, n_req, 16, 48, second, req_dim)
    rows, mask = _oracle(wl)
    brows, bmask = _brute(wl)
    assert np.array_equal(mask, bmask)
    if len(mask):
        assert rows.shape == brows.shape
        assert np.array_equal(rows, brows)
    if second:  # ignoring the engager slots must reproduce the first-degree result
        r1, m1 = _oracle(wl, first_degree_only=True)
        b1, bm1 = _brute(wl, first_degree_only=True)
        assert np.array_equal(m1, bm1) and (len(m1) == 0 or np.array_equal(r1, b1))
        assert np.array_equal(m1, mask & 1)


# ---------------------------------------------------------------- Algorithm 1 with library ops
def _alg1_torch(keys, feats, d):
    """Steps 2-4 of Algorithm 1 for one request, restated with the library ops the paper names."""
    K = keys.shape[0]
    if K == 0:
        return torch.zeros((d.shape[0], feats.shape[1]), dtype=feats.dtype), torch.zeros(d.shape[0], dtype=torch.bool)
    pos = torch.searchsorted(keys, d, right=False)
    pos_safe = torch.clamp(pos, max=K - 1)
    valid = (pos < K) & (keys[pos_safe] == d)
    O = torch.zeros((d.shape[0], feats.shape[1]), dtype=feats.dtype)
    O[valid] = feats.index_select(0, pos_safe[valid])
    return O, valid


@pytest.mark.parametrize("maker", [
    lambda: W.config0(n_docs=20_000, n_cand=6_000, k=500),
    lambda: W.config1(n_docs=40_000, n_req=6, n_cand=3_000),
])
def test_oracle_equals_algorithm1_library_ops(maker):
    wl = maker()
    s, b = wl.store, wl.batch
    rows, mask = _oracle(wl)
    doc_b, edge_b = s.doc_row_bytes, b.edge_row_bytes
    for r in range(b.n_req):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        d = torch.from_numpy(s.author_ids[b.cand_idx[c0:c1].astype(np.int64)])
        O, valid = _alg1_torch(torch.from_numpy(b.edge_keys[e0:e1]),
                               torch.from_numpy(b.edge_feats[e0:e1].view(np.int16)), d)
        got = rows[c0:c1, doc_b:doc_b + edge_b].copy().view(np.int16)
        assert np.array_equal(got, O.numpy())
        assert np.array_equal(mask[c0:c1], valid.numpy().astype(np.uint8))
        # doc section is a plain gather by position, request section a broadcast
        gathered = torch.from_numpy(s.doc_feats.view(np.uint8).reshape(s.n_docs, -1)).index_select(
            0, torch.from_numpy(b.cand_idx[c0:c1].astype(np.int64))).numpy()
        assert np.array_equal(rows[c0:c1, :doc_b], gathered)
        if b.req_feats is not None:
            want = np.broadcast_to(b.req_feats[r].view(np.uint8), (c1 - c0, b.req_row_bytes))
            assert np.array_equal(rows[c0:c1, doc_b + edge_b:], want)


# ---------------------------------------------------------------- the paper's worked example
def test_worked_batching_example_from_the_paper():
    req, flat = [], None
    for line in open(os.path.join(GOLDEN, "batching_example.txt")):
        if line.startswith("request"):
            req.append([int(x) for x in line.split(":")[1].split()])
        elif line.startswith("flattened"):
            flat = [int(x) for x in line.split(":")[1].split()]
    assert flat == sum(req, [])
    rng = np.random.default_rng(1)
    store = W.make_store(rng, 100, 50, 8, np.float32, tagged=True)
    keys, feats = W.make_viewer(rng, 50, 5, 8, np.float16)
    batch = W.assemble_batch([keys, keys], [feats, feats], [np.array(x, np.int32) for x in req], None,
                             8, np.float16, 0, np.float32)
    rows, _ = _oracle(W.Workload("example", 1, store, batch))
    doc_b = store.doc_row_bytes
    assert list(batch.cand_offsets) == [0, 3, 5]
    for k, p in enumerate(flat):
        assert np.array_equal(rows[k, :doc_b], store.doc_feats[p].view(np.uint8))
        # tagged store: the first value of row p is p * doc_dim
        assert rows[k, :4].copy().view(np.float32)[0] == (p * 8) % 2048


def _read_golden_example():
    req, flat, scatter, T = [], None, None, []
    for line in open(os.path.join(GOLDEN, "batching_example.txt")):
        if line.startswith("request"):
            req.append([int(x) for x in line.split(":")[1].split()])
        elif line.startswith("flattened"):
            flat = [int(x) for x in line.split(":")[1].split()]
        elif line.startswith("scatter"):
            scatter = [tuple(int(v) for v in x.split(",")) for x in line.split(":")[1].split()]
        elif line.startswith("T "):
            T.append([None if x == "pad" else int(x) for x in line.split(":")[1].split()])
    return req, flat, scatter, T


def _example_workload(cands, n_docs=100):
    rng = np.random.default_rng(1)
    store = W.make_store(rng, n_docs, 50, 8, np.float32, tagged=True)
    keys, feats = W.make_viewer(rng, 50, 5, 8, np.float16)
    batch = W.assemble_batch([keys] * len(cands), [feats] * len(cands), [np.array(x, np.int32) for x in cands], None,
                             8, np.float16, 0, np.float32)
    return W.Workload("example", 1, store, batch)


def _padded(wl, n_max=None, **kw):
    s, b = wl.store, wl.batch
    return oracle.join_padded(
        s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets, n_max=n_max,
        req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types, reduce_sum_mask=s.reduce_sum_mask, **kw)


def test_padded_layout_of_the_worked_example():
    """The scatter indices and the padded tensor T the paper prints for its b = 2 example."""
    req, flat, scatter, T = _read_golden_example()
    wl = _example_workload(req)
    s, b = wl.store, wl.batch
    valid, batch_idx, pos_idx = oracle.scatter_indices(b.cand_idx, b.cand_offsets, s.n_docs)
    assert valid.all() and list(zip(batch_idx.tolist(), pos_idx.tolist())) == scatter
    out, mask, n_valid, src = _padded(wl)
    assert out.shape[:2] == (2, 3) and list(n_valid) == [3, 2] and list(src) == [0, 1, 2, 3, 4]
    doc_b = s.doc_row_bytes
    for r, line in enumerate(T):
        for k, p in enumerate(line):
            if p is None:  # the pad
                assert not out[r, k].any() and mask[r, k] == 0
            else:
                assert np.array_equal(out[r, k, :doc_b], s.doc_feats[p].view(np.uint8))
                assert out[r, k, :4].copy().view(np.float32)[0] == (p * 8) % 2048  # tagged store: row p starts with p * 8


def test_padded_layout_drops_unresolved_positions_by_hand():
    """Same example with unresolved (-1) and out-of-range positions mixed in: they get no scatter index, the
    valid ones close ranks in their input order.  Expected values written out by hand."""
    wl = _example_workload([[-1, 10, 42, -1, 87], [100, 5, -1, 63], [-1, -1], []])
    s, b = wl.store, wl.batch
    valid, batch_idx, pos_idx = oracle.scatter_indices(b.cand_idx, b.cand_offsets, s.n_docs)
    assert valid.tolist() == [False, True, True, False, True, False, True, False, True, False, False]
    assert list(zip(batch_idx.tolist(), pos_idx.tolist())) == [(0, 0), (0, 1), (0, 2), (1, 0), (1, 1)]
    out, mask, n_valid, src = _padded(wl)
    assert out.shape[:2] == (4, 3) and list(n_valid) == [3, 2, 0, 0] and list(src) == [1, 2, 4, 6, 8]
    want = [[10, 42, 87], [5, 63, None], [None] * 3, [None] * 3]
    for r in range(4):
        for k in range(3):
            if want[r][k] is None:
                assert not out[r, k].any() and mask[r, k] == 0
            else:
                assert out[r, k, :4].copy().view(np.float32)[0] == (want[r][k] * 8) % 2048
    # a wider n_max only adds pads; a narrower one drops the tail of the longer requests
    wide, wmask, _, _ = _padded(wl, n_max=5)
    assert np.array_equal(wide[:, :3], out) and not wide[:, 3:].any() and not wmask[:, 3:].any()
    narrow, nmask, _, _ = _padded(wl, n_max=2)
    assert np.array_equal(narrow, out[:, :2]) and np.array_equal(nmask, mask[:, :2])


@settings(max_examples=40, deadline=None, suppress_health_check=list(HealthCheck))
@given(seed=st.integers(0, 2**31), n_docs=st.integers(1, 40), alphabet=st.integers(1, 24),
       n_req=st.integers(0, 4), second=st.booleans(), req_dim=st.sampled_from([0, 4]))
def test_padded_equals_naive_scan_rows_placed_one_by_one(seed, n_docs, alphabet, n_req, second, req_dim):
    """Compaction before the join (the oracle's route) against the naive scan over the uncompacted batch whose
    valid rows are then placed one at a time."""
    wl = _tiny(seed, n_docs, alphabet, n_req, 16, 48, second, req_dim)
    s, b = wl.store, wl.batch
    out, mask, n_valid, src = _padded(wl)
    brows, bmask = _brute(wl)
    assert out.shape[0] == b.n_req
    kept = []
    for r in range(b.n_req):
        k = 0
        for j in range(int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])):
            if 0 <= int(b.cand_idx[j]) < s.n_docs:
                assert np.array_equal(out[r, k], brows[j]) and mask[r, k] == bmask[j]
                kept.append(j)
                k += 1
        assert k == n_valid[r]
        assert not out[r, k:].any() and not mask[r, k:].any()
    assert kept == list(src)


# ---------------------------------------------------------------- invariants at realistic shapes
def _check_invariants(wl):
    s, b = wl.store, wl.batch
    rows, mask = _oracle(wl)
    doc_b, edge_b, req_b = s.doc_row_bytes, b.edge_row_bytes, b.req_row_bytes
    assert rows.shape == (b.total_cands, wl.out_row_bytes())
    docs_u8 = s.doc_feats.view(np.uint8).reshape(s.n_docs, -1)
    edge_u8 = b.edge_feats.view(np.uint8).reshape(len(b.edge_keys), -1)
    for r in range(b.n_req):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        keyset = {int(k): i for i, k in enumerate(b.edge_keys[e0:e1])}
        cand = b.cand_idx[c0:c1].astype(np.int64)
        auth = s.author_ids[cand]
        member = np.array([int(a) in keyset for a in auth], dtype=bool)
        # found count = size of the intersection (as a multiset over candidates)
        assert int((mask[c0:c1] & 1).sum()) == int(member.sum())
        assert np.array_equal((mask[c0:c1] & 1).astype(bool), member)
        # every row is the concatenation of its source rows (or zeros)
        assert np.array_equal(rows[c0:c1, :doc_b], docs_u8[cand])
        src = np.array([keyset.get(int(a), 0) for a in auth]) + e0
        want_edge = np.where(member[:, None], edge_u8[src], 0)
        assert np.array_equal(rows[c0:c1, doc_b:doc_b + edge_b], want_edge)
        if req_b:
            assert np.all(rows[c0:c1, -req_b:] == b.req_feats[r].view(np.uint8)[None, :])
    return rows, mask


def test_invariants_config0_full_size():
    wl = W.config0()
    assert wl.batch.total_cands == 20_000 and wl.batch.max_edge_len == 500
    assert wl.out_row_bytes() == 320
    assert len(np.unique(wl.batch.cand_idx)) == 20_000  # drawn without replacement
    rows, mask = _check_invariants(wl)
    frac = float((mask & 1).mean())
    assert 0.69 < frac < 0.72, frac  # 70 % forced plus a few chance hits


def test_invariants_config1_scaled():
    wl = W.config1(n_docs=60_000, n_req=8, n_cand=4_000)
    assert wl.out_row_bytes() == 384
    _check_invariants(wl)


def test_batch_equals_single_requests_and_permutation_equivariance():
    wl = W.config1(n_docs=30_000, n_req=5, n_cand=700)
    s, b = wl.store, wl.batch
    rows, mask = _oracle(wl)
    for r in range(b.n_req):
        e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        one = W.assemble_batch([b.edge_keys[e0:e1]], [b.edge_feats[e0:e1]], [b.cand_idx[c0:c1]],
                               b.req_feats[r:r + 1], b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype)
        r1, m1 = _oracle(W.Workload("one", 0, s, one))
        assert np.array_equal(r1, rows[c0:c1]) and np.array_equal(m1, mask[c0:c1])
    perm = np.random.default_rng(0).permutation(int(b.cand_offsets[1]))
    cand2 = b.cand_idx.copy()
    cand2[: len(perm)] = b.cand_idx[: len(perm)][perm]
    r2, m2 = _oracle(W.Workload("perm", 0, s, W.Batch(**{**b.__dict__, "cand_idx": cand2})))
    assert np.array_equal(r2[: len(perm)], rows[: len(perm)][perm])
    assert np.array_equal(m2[: len(perm)], mask[: len(perm)][perm])
    assert np.array_equal(r2[len(perm):], rows[len(perm):])
    # a threaded run partitions candidates only
    r3, m3 = _oracle(wl, n_threads=3)
    assert np.array_equal(r3, rows) and np.array_equal(m3, mask)


# ---------------------------------------------------------------- boundary cases of Algorithm 1 step 3
def test_search_boundaries():
    imax = np.iinfo(np.int64).max
    author_ids = np.array([0, 5, 7, 9, imax, imax - 1, -3, 6], dtype=np.int64)
    docs = np.arange(8 * 4, dtype=np.float32).reshape(8, 4)
    keys = np.array([0, 7, imax], dtype=np.int64)
    feats = np.array([[1, 2], [3, 4], [5, 6]], dtype=np.float16)
    cand = np.array([0, 1, 2, 3, 4, 5, 6, 7, 2, 2, -1, 8], dtype=np.int32)
    rows, mask = oracle.join(docs, author_ids, keys, feats, np.array([0, 3]), cand, np.array([0, len(cand)]))
    assert list(mask) == [1, 0, 1, 0, 1, 0, 0, 0, 1, 1, 0, 0]
    edge = rows[:, 16:].copy().view(np.float16)
    assert edge.tolist() == [[1, 2], [0, 0], [3, 4], [0, 0], [5, 6], [0, 0], [0, 0], [0, 0], [3, 4], [3, 4], [0, 0], [0, 0]]
    assert not rows[10].any() and not rows[11].any()  # unresolved / out-of-range position: zero row
    # K == 0 and K == 1
    r0, m0 = oracle.join(docs, author_ids, keys[:0], feats[:0], np.array([0, 0]), cand, np.array([0, len(cand)]))
    assert not m0.any() and not r0[:, 16:].any()
    r1, m1 = oracle.join(docs, author_ids, keys[1:2], feats[1:2], np.array([0, 1]), cand, np.array([0, len(cand)]))
    assert list(m1) == [0, 0, 1, 0, 0, 0, 0, 0, 1, 1, 0, 0]
    # requests with no candidates in the middle of a batch
    r2, m2 = oracle.join(docs, author_ids, np.concatenate([keys, keys]), np.concatenate([feats, feats]),
                         np.array([0, 3, 3, 6]), cand, np.array([0, 0, 5, len(cand)]))
    assert list(m2) == [0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 0, 0]


# ---------------------------------------------------------------- second-degree reduction (unpinned by the paper)
def _second_case(actor_rows, types, keys, feats, sum_mask, author=999):
    n = len(actor_rows)
    docs = np.zeros((n, 2), dtype=np.float32)
    author_ids = np.full(n, author, dtype=np.int64)
    return oracle.join(docs, author_ids, np.asarray(keys, np.int64), np.asarray(feats, np.float16),
                       np.array([0, len(keys)]), np.arange(n, dtype=np.int32), np.array([0, n]),
                       actor_ids=np.asarray(actor_rows, np.int64), actor_types=np.asarray(types, np.uint8),
                       reduce_sum_mask=sum_mask)


def test_second_degree_special_cases():
    keys = [10, 20, 30, 40]
    feats = [[1.0, 8.0, -1.0, 2.0], [3.0, 0.5, -4.0, 2.0], [2.0, 0.25, -0.0, 2.0], [0.5, 100.0, 5.0, 2.0]]
    actors = [[-1, -1, -1, -1],      # nothing to look up
              [11, 21, -1, -1],      # engagers present, none is a key
              [-1, 30, -1, -1],      # exactly one found: edge2 is that row, bit for bit, for max and for sum
              [10, 20, 30, 40],      # all four found
              [40, 20, 40, 5],       # a key found twice is counted twice; slot 3 misses
              [20, 10, -1, -1]]      # order of slots is the order of reduction
    types = [[0, 0, 0, 0], [1, 2, 0, 0], [0, 2, 0, 0], [0, 1, 2, 0], [1, 1, 1, 2], [2, 2, 0, 0]]
    sum_mask = 0b1010  # dims 1 and 3 summed, dims 0 and 2 max
    rows, mask = _second_case(actors, types, keys, feats, sum_mask)
    e1 = rows[:, 8:16].copy().view(np.float16)
    e2 = rows[:, 16:24].copy().view(np.float16)
    assert not e1.any()  # author 999 is not a key
    assert list(mask) == [0, 0, 0b10000100, 0b11111110, 0b01001110, 0b10000110]
    assert e2[0].tolist() == [0, 0, 0, 0] and e2[1].tolist() == [0, 0, 0, 0]
    # one found slot: bit-identical copy (the -0.0 in a max dim keeps its sign bit)
    assert np.array_equal(e2[2].view(np.uint16), np.asarray(feats[2], np.float16).view(np.uint16))
    assert e2[3].tolist() == [3.0, 108.75, 5.0, 8.0]
    assert e2[4].tolist() == [3.0, 200.5, 5.0, 6.0]
    assert e2[5].tolist() == [3.0, 8.5, -1.0, 4.0]


def test_second_degree_sum_matches_float64_when_partial_sums_are_exact():
    rng = np.random.default_rng(11)
    K, n = 64, 500
    keys = np.arange(0, 2 * K, 2)
    feats = rng.integers(-64, 65, size=(K, 8)).astype(np.float16)  # small integers: every fp32 partial sum is exact
    actors = rng.integers(0, 2 * K, size=(n, 4))
    actors[rng.random((n, 4)) < 0.2] = -1
    types = rng.integers(0, 3, size=(n, 4))
    rows, mask = _second_case(actors, types, keys, feats, 0xFF)
    e2 = rows[:, 8 + 16: 8 + 32].copy().view(np.float16)
    for j in range(n):
        hit = [int(a) // 2 for a in actors[j] if a >= 0 and a % 2 == 0]
        want = np.zeros(8) if not hit else feats[hit].astype(np.float64).sum(axis=0)
        assert np.array_equal(e2[j].astype(np.float64), want)
        bits = sum(1 << (1 + s) for s, a in enumerate(actors[j]) if a >= 0 and a % 2 == 0)
        assert (int(mask[j]) & 0b11110) == bits


def test_second_degree_max_is_an_input_and_dominates():
    rng = np.random.default_rng(12)
    K, n = 40, 400
    keys = np.arange(K)
    feats = rng.standard_normal((K, 8)).astype(np.float16)
    actors = rng.integers(-1, K + 10, size=(n, 4))
    rows, mask = _second_case(actors, np.zeros((n, 4)), keys, feats, 0)
    e2 = rows[:, 8 + 16: 8 + 32].copy().view(np.float16)
    for j in range(n):
        hit = [int(a) for a in actors[j] if 0 <= a < K]
        if not hit:
            assert not e2[j].any()
            continue
        assert np.array_equal(e2[j], feats[hit].max(axis=0))


def test_generators_are_deterministic():
    a = W.config1(n_docs=20_000, n_req=3, n_cand=500)
    b = W.config1(n_docs=20_000, n_req=3, n_cand=500)
    for x, y in ((a.store.author_ids, b.store.author_ids), (a.store.doc_feats, b.store.doc_feats),
                 (a.batch.edge_keys, b.batch.edge_keys), (a.batch.cand_idx, b.batch.cand_idx)):
        assert W.checksum64(x) == W.checksum64(y)
    for r in range(3):
        k = a.batch.edge_keys[a.batch.edge_offsets[r]:a.batch.edge_offsets[r + 1]]
        assert np.all(np.diff(k) > 0)


@pytest.mark.timeout(60)
def test_generator_refuses_more_distinct_candidates_than_documents():
    # a request cannot draw more distinct documents than the store holds: an error, not an endless rejection loop
    with pytest.raises(ValueError):
        W.config1(n_docs=5_754, n_req=3, n_cand=8_134, second_degree=True, edge_lo=37, edge_hi=5_164)


# ---------------------------------------------------------------- Algorithm 1 step 1 (sort of the affinity records)
def _unsorted_batch(seed, n_req, kmax, alphabet, dup=False):
    rng = np.random.default_rng(seed)
    keys_l, feats_l = [], []
    for _ in range(n_req):
        k = int(rng.integers(0, kmax + 1))
        keys = rng.integers(0, alphabet, size=k) if dup else rng.permutation(alphabet)[:k]
        keys_l.append(keys.astype(np.int64))
        feats_l.append(rng.standard_normal((k, 8)).astype(np.float16))
    eo = np.concatenate([[0], np.cumsum([len(k) for k in keys_l])]).astype(np.int64)
    return np.concatenate(keys_l + [np.empty(0, np.int64)]), np.concatenate(feats_l + [np.empty((0, 8), np.float16)]), eo


@pytest.mark.parametrize("dup", [False, True])
def test_sort_step_matches_library_sort_and_gather(dup):
    keys, feats, eo = _unsorted_batch(3 + dup, n_req=9, kmax=300, alphabet=200 if dup else 5000, dup=dup)
    ks, fs, perm = oracle.sort_edges(keys, feats, eo)
    for r in range(len(eo) - 1):
        a, z = int(eo[r]), int(eo[r + 1])
        # numpy's stable argsort, and Algorithm 1 step 1 restated with torch.sort(stable=True) + gather
        order = np.argsort(keys[a:z], kind="stable")
        assert np.array_equal(perm[a:z], order)
        assert np.array_equal(ks[a:z], keys[a:z][order])
        assert np.array_equal(fs[a:z].view(np.uint16), feats[a:z][order].view(np.uint16))
        tk, tidx = torch.sort(torch.from_numpy(keys[a:z]), stable=True)
        assert np.array_equal(tk.numpy(), ks[a:z]) and np.array_equal(tidx.numpy(), perm[a:z])
        assert np.all(np.diff(ks[a:z]) >= 0)
        assert sorted(perm[a:z].tolist()) == list(range(z - a))


def test_join_after_sort_equals_naive_scan_on_unsorted_records():
    """Eq. 1 does not ask for sorted records: the naive scan on the *unsorted* (a, F) must equal the join of
    the records sorted by Algorithm 1 step 1 (unique keys)."""
    wl = tiny_workload(21, n_docs=60, alphabet=40, n_req=4, kmax=25, nmax=50, second=False, req_dim=4)
    b, s = wl.batch, wl.store
    rng = np.random.default_rng(2)
    keys_u, feats_u = b.edge_keys.copy(), b.edge_feats.copy()
    for r in range(b.n_req):
        a, z = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        p = rng.permutation(z - a)
        keys_u[a:z], feats_u[a:z] = b.edge_keys[a:z][p], b.edge_feats[a:z][p]
    ks, fs, _ = oracle.sort_edges(keys_u, feats_u, b.edge_offsets)
    assert np.array_equal(ks, b.edge_keys) and np.array_equal(fs.view(np.uint16), b.edge_feats.view(np.uint16))
    rows, mask = oracle.join(s.doc_feats, s.author_ids, ks, fs, b.edge_offsets, b.cand_idx, b.cand_offsets, req_feats=b.req_feats)
    brows, bmask = brute_force.join(s.doc_feats, s.author_ids, keys_u, feats_u, b.edge_offsets, b.cand_idx, b.cand_offsets,
                                    req_feats=b.req_feats)
    assert np.array_equal(mask, bmask) and np.array_equal(rows, brows)


# ---------------------------------------------------------------- Eq. 6 (document id -> position)
def test_id_resolution_matches_a_hash_map_and_searchsorted():
    rng = np.random.default_rng(8)
    ids = np.cumsum(rng.integers(1, 9, size=5000)).astype(np.int64) * 2  # ascending, unique, even
    positions = rng.permutation(len(ids)).astype(np.int32)
    present = ids[rng.integers(0, len(ids), size=3000)]
    absent = np.concatenate([present[:500] + 1, [ids[0] - 2, ids[-1] + 2, -5, np.iinfo(np.int64).max]])
    q = np.concatenate([present, absent])
    rng.shuffle(q)
    H = {int(k): int(p) for k, p in zip(ids, positions)}  # the paper's CPU design: a hash map
    want = np.array([H.get(int(x), -1) for x in q], dtype=np.int32)
    assert np.array_equal(oracle.resolve_ids(ids, q, positions), want)
    rank = np.searchsorted(ids, q)
    hit = (rank < len(ids)) & (ids[np.minimum(rank, len(ids) - 1)] == q)
    assert np.array_equal(oracle.resolve_ids(ids, q), np.where(hit, rank, -1).astype(np.int32))
    assert np.array_equal(oracle.resolve_ids(ids[:0], q), np.full(len(q), -1, np.int32))


# ---------------------------------------------------------------- store write path (Section 6.2, ingestion step 3)
def test_upsert_closed_forms():
    rng = np.random.default_rng(3)
    n, d = 57, 6
    X = rng.standard_normal((n, d)).astype(np.float32)
    ids = rng.integers(0, 1000, size=n, dtype=np.int64)
    act = rng.integers(-1, 50, size=(n, 4), dtype=np.int64)
    typ = rng.integers(0, 3, size=(n, 4)).astype(np.uint8)
    # a batch that names every row once, positions = a permutation pi: the result is the batch read through pi^-1
    pi = rng.permutation(n)
    newX = rng.standard_normal((n, d)).astype(np.float32)
    newids = rng.integers(0, 1000, size=n, dtype=np.int64)
    newact = rng.integers(-1, 50, size=(n, 4), dtype=np.int64)
    newtyp = rng.integers(0, 3, size=(n, 4)).astype(np.uint8)
    X0, ids0 = X.copy(), ids.copy()
    Y, yid, yact, ytyp = oracle.upsert(X, ids, pi, newX, newids, act, typ, newact, newtyp)
    inv = np.argsort(pi)
    assert np.array_equal(Y, newX[inv]) and np.array_equal(yid, newids[inv])
    assert np.array_equal(yact, newact[inv]) and np.array_equal(ytyp, newtyp[inv])
    assert np.array_equal(X, X0) and np.array_equal(ids, ids0) and not np.shares_memory(Y, X)  # inputs are not modified
    # a partial batch: named rows change, all others keep their old content; out-of-range positions write nothing
    pos = np.array([5, -1, 56, n, 0, 2**31 - 1, 17], dtype=np.int64)
    Z, zid, zact, ztyp = oracle.upsert(X, ids, pos, newX[:7], newids[:7], act, typ, newact[:7], None)
    keep = np.ones(n, dtype=bool)
    for i, p in [(0, 5), (2, 56), (4, 0), (6, 17)]:
        assert np.array_equal(Z[p], newX[i]) and zid[p] == newids[i] and np.array_equal(zact[p], newact[i])
        keep[p] = False
    assert np.array_equal(Z[keep], X[keep]) and np.array_equal(zid[keep], ids[keep]) and np.array_equal(zact[keep], act[keep])
    assert np.array_equal(ztyp, typ)  # no new types given: untouched everywhere
    # the same batch twice = once; batches over disjoint rows commute; the empty batch is the identity
    Z2 = oracle.upsert(Z, zid, pos, newX[:7], newids[:7], zact, ztyp, newact[:7], None)
    assert all(np.array_equal(a, b) for a, b in zip(Z2, (Z, zid, zact, ztyp)))
    a_pos, b_pos = np.array([1, 2, 3]), np.array([40, 41])
    ab = oracle.upsert(*oracle.upsert(X, ids, a_pos, newX[:3], newids[:3])[:2], b_pos, newX[3:5], newids[3:5])
    ba = oracle.upsert(*oracle.upsert(X, ids, b_pos, newX[3:5], newids[3:5])[:2], a_pos, newX[:3], newids[:3])
    assert np.array_equal(ab[0], ba[0]) and np.array_equal(ab[1], ba[1])
    E = oracle.upsert(X, ids, np.empty(0, np.int64), newX[:0], newids[:0])
    assert np.array_equal(E[0], X) and np.array_equal(E[1], ids)
    with pytest.raises(ValueError):
        oracle.upsert(X, ids, np.array([4, 4]), newX[:2], newids[:2])


def test_join_sees_upserted_rows_like_a_store_built_directly():
    """Join after an upsert = naive scan over a store that was generated with the final contents."""
    wl = _tiny(77, 30, 12, 3, 10, 40, True, 4)
    s = wl.store
    rng = np.random.default_rng(8)
    pos = rng.permutation(s.n_docs)[:11]
    donor = W.make_store(np.random.default_rng(99), s.n_docs, 12, 4, np.float32, max_actors=4, reduce_sum_mask=s.reduce_sum_mask)
    doc, auth, act, typ = oracle.upsert(s.doc_feats, s.author_ids, pos, donor.doc_feats[pos], donor.author_ids[pos],
                                        s.actor_ids, s.actor_types, donor.actor_ids[pos], donor.actor_types[pos])
    # built directly: donor rows where named, original rows elsewhere, chosen row by row
    named = set(int(p) for p in pos)
    for arr_new, arr_old, arr_don in ((doc, s.doc_feats, donor.doc_feats), (auth, s.author_ids, donor.author_ids),
                                      (act, s.actor_ids, donor.actor_ids), (typ, s.actor_types, donor.actor_types)):
        for p in range(s.n_docs):
            assert np.array_equal(arr_new[p], arr_don[p] if p in named else arr_old[p])
    b = wl.batch
    rows, mask = oracle.join(doc, auth, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets,
                             req_feats=b.req_feats, actor_ids=act, actor_types=typ, reduce_sum_mask=s.reduce_sum_mask)
    brows, bmask = brute_force.join(doc, auth, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets,
                                    req_feats=b.req_feats, actor_ids=act, actor_types=typ,
                                    reduce_sum_mask=s.reduce_sum_mask)
    assert np.array_equal(rows, brows) and np.array_equal(mask, bmask)


# ---------------------------------------------------------------- derived features (Section 4.1.2): chunked cosine
def _f16_ulp(v):
    """Spacing of float16 at |v| (subnormal spacing below the smallest normal)."""
    a = np.maximum(np.abs(np.asarray(v, dtype=np.float64)), 2.0 ** -14)
    return 2.0 ** (np.floor(np.log2(a)) - 10)


def _cos_case(seed, n_docs=200, doc_dim=64, item_first=8, dim=50, n_chunks=3, n_req=3, n_cand=40, scale=1.0):
    rng = np.random.default_rng(seed)
    docs = (scale * rng.standard_normal((n_docs, doc_dim))).astype(np.float16)
    member = (scale * rng.standard_normal((n_req, n_chunks * dim))).astype(np.float16)
    cands = [rng.integers(-1, n_docs + 1, size=int(rng.integers(0, n_cand + 1))).astype(np.int32) for _ in range(n_req)]
    co = np.concatenate([[0], np.cumsum([len(c) for c in cands])]).astype(np.int64)
    return docs, member, np.concatenate(cands).astype(np.int32), co


@pytest.mark.parametrize("seed,dim,n_chunks,item_first,scale", [(0, 50, 3, 8, 1.0), (1, 50, 3, 0, 30.0), (2, 7, 1, 16, 0.01),
                                                                (3, 64, 4, 0, 1.0), (4, 1, 8, 56, 1.0)])
def test_cosine_against_float64_and_a_numpy_float32_restatement(seed, dim, n_chunks, item_first, scale):
    docs, member, ci, co = _cos_case(seed, dim=dim, n_chunks=n_chunks, item_first=item_first, scale=scale)
    got = oracle.cosine_features(docs, member, ci, co, item_first, dim, n_chunks)
    assert got.shape == (len(ci), 32)
    vals = got.copy().view(np.float16).astype(np.float64)  # [C, 16]
    assert not vals[:, n_chunks:].any()
    req_of = np.searchsorted(co, np.arange(len(ci)), side="right") - 1
    ok = (ci >= 0) & (ci < docs.shape[0])
    x = np.where(ok[:, None], docs[np.where(ok, ci, 0), item_first:item_first + dim], 0)
    # (a) the mathematical definition in float64: within one float16 spacing + the float32 accumulation error
    x64 = x.astype(np.float64)
    for k in range(n_chunks):
        m64 = member[req_of, k * dim:(k + 1) * dim].astype(np.float64)
        den = np.linalg.norm(x64, axis=1) * np.linalg.norm(m64, axis=1)
        want = np.where(den > 1e-8, (x64 * m64).sum(axis=1) / np.maximum(den, 1e-8), 0.0)
        assert np.all(np.abs(vals[:, k] - want) <= _f16_ulp(want) * 0.5001 + 1e-5), k
    # (b) bit for bit: float16 x float16 products are exact in float32, so the fused chain equals a plain float32
    #     multiply-add chain, written here with numpy float32 ops over all candidates at once
    x32 = x.astype(np.float32)
    nx = np.zeros(len(ci), np.float32)
    for e in range(dim):
        nx = nx + x32[:, e] * x32[:, e]
    for k in range(n_chunks):
        m32 = member[req_of, k * dim:(k + 1) * dim].astype(np.float32)
        dot, nm = np.zeros(len(ci), np.float32), np.zeros(len(ci), np.float32)
        for e in range(dim):
            dot = dot + x32[:, e] * m32[:, e]
            nm = nm + m32[:, e] * m32[:, e]
        den = np.sqrt(nx) * np.sqrt(nm)
        den = np.where(den > np.float32(1e-8), den, np.float32(1e-8)).astype(np.float32)
        with np.errstate(over="ignore"):
            want16 = (dot / den).astype(np.float16)
        assert np.array_equal(got[:, 2 * k:2 * k + 2].copy().view(np.uint16)[:, 0], want16.view(np.uint16)), k


def test_cosine_closed_forms():
    dim, n_chunks, first = 50, 3, 8
    rng = np.random.default_rng(9)
    base = rng.standard_normal(dim).astype(np.float16)
    base[base == 0] = np.float16(0.5)
    ortho_a = np.zeros(dim, np.float16); ortho_a[3] = 2.0
    ortho_b = np.zeros(dim, np.float16); ortho_b[4] = -7.0
    docs = np.zeros((6, 64), np.float16)
    docs[:, :first] = 9.0          # other document features around the embedding must not leak in
    docs[:, first + dim:] = -9.0
    docs[0, first:first + dim] = base                  # same direction as medoid 0
    docs[1, first:first + dim] = -base                 # opposite
    docs[2, first:first + dim] = base * np.float16(2)  # scaled (exact in float16)
    docs[3, first:first + dim] = ortho_a               # orthogonal to medoid 1
    docs[4, first:first + dim] = 0                     # zero item embedding
    docs[5, first:first + dim] = base
    member = np.zeros((2, n_chunks * dim), np.float16)
    member[0, 0:dim] = base
    member[0, dim:2 * dim] = ortho_b
    member[0, 2 * dim:] = base * np.float16(-0.5)
    member[1] = 0                                      # a request with an all-zero member representation
    ci = np.array([0, 1, 2, 3, 4, -1, 6, 5], np.int32)
    co = np.array([0, 7, 8], np.int64)
    v = oracle.cosine_features(docs, member, ci, co, first, dim, n_chunks).copy().view(np.float16).reshape(-1, 16)
    one, minus = np.float16(1.0), np.float16(-1.0)
    assert v[0, 0] == one and v[0, 2] == minus           # parallel / anti-parallel
    assert v[1, 0] == minus and v[1, 2] == one
    assert v[2, 0] == one and v[2, 2] == minus           # scale invariance
    assert v[3, 1] == 0 and v[0, 1] != 0                 # orthogonal unit directions
    assert not v[4].any() and not v[5].any() and not v[6].any()  # zero item, unresolved (-1) and out-of-range position
    assert not v[7].any()                                # zero member representation
    assert not v[:, n_chunks:].any()
    # NaN is stored as 0x7fff: an infinite component makes |x| infinite and the quotient inf / inf
    docs[0, first] = np.float16(np.inf)
    w = oracle.cosine_features(docs, member, ci[:1], np.array([0, 1, 1], np.int64), first, dim, n_chunks)
    assert w.copy().view(np.uint16)[0, 0] == 0x7FFF
