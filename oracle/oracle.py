"""TEST INFRASTRUCTURE — Python entry to the CPU oracle (oracle/ccr_oracle.cpp).

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may import this.
It does not import the product package and the product package never imports it; the oracle
takes plain numpy arrays (or any object with the attribute names used below).

`build()` compiles the C++ with g++ into oracle/libccr_oracle.so (building the checker is not
using it); `join(...)` runs Eq. 1 / Algorithm 1 steps 2-4 of the paper plus the doc-row gather and
request broadcast for a ragged batch and returns (out_rows uint8[C, out_b], out_mask uint8[C]).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ccr_oracle.cpp")
_LIB = os.path.join(_HERE, "libccr_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    with _lock:
        stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, i32, u64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint64
        lib.ccr_oracle_join.restype = ctypes.c_int
        lib.ccr_oracle_join.argtypes = [
            i64, vp, i64, vp, i32, vp, vp, i32, i32, u64,
            i32, vp, vp, vp, vp, vp, vp, i64, i32, vp, vp, i32,
        ]
        lib.ccr_oracle_resolve_ids.restype = ctypes.c_int
        lib.ccr_oracle_resolve_ids.argtypes = [i64, vp, vp, i64, vp, vp]
        lib.ccr_oracle_sort_edges.restype = ctypes.c_int
        lib.ccr_oracle_sort_edges.argtypes = [i32, vp, vp, vp, i64, vp, vp, vp]
        lib.ccr_oracle_cosine.restype = ctypes.c_int
        lib.ccr_oracle_cosine.argtypes = [i64, vp, i64, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.ccr_oracle_half_to_float_bits.restype = ctypes.c_uint32
        lib.ccr_oracle_half_to_float_bits.argtypes = [ctypes.c_uint16]
        lib.ccr_oracle_float_bits_to_half.restype = ctypes.c_uint16
        lib.ccr_oracle_float_bits_to_half.argtypes = [ctypes.c_uint32]
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def out_row_bytes(doc_feats, edge_feats, req_feats, max_actors: int, first_degree_only: bool) -> int:
    doc_b = doc_feats.shape[1] * doc_feats.dtype.itemsize
    edge_b = edge_feats.shape[1] * edge_feats.dtype.itemsize
    req_b = 0 if req_feats is None else req_feats.shape[1] * req_feats.dtype.itemsize
    second = max_actors > 0 and not first_degree_only
    return doc_b + edge_b + (edge_b if second else 0) + req_b


def join(
    doc_feats: np.ndarray,
    author_ids: np.ndarray,
    edge_keys: np.ndarray,
    edge_feats: np.ndarray,
    edge_offsets: np.ndarray,
    cand_idx: np.ndarray,
    cand_offsets: np.ndarray,
    req_feats: Optional[np.ndarray] = None,
    actor_ids: Optional[np.ndarray] = None,
    actor_types: Optional[np.ndarray] = None,
    reduce_sum_mask: int = 0,
    first_degree_only: bool = False,
    n_threads: int = 1,
) -> Tuple[np.ndarray, np.ndarray]:
    lib = _load()
    doc_feats = _c(doc_feats)
    author_ids = _c(author_ids, np.int64)
    edge_keys = _c(edge_keys, np.int64)
    edge_feats = _c(edge_feats)
    edge_offsets = _c(edge_offsets, np.int64)
    cand_idx = _c(cand_idx, np.int32)
    cand_offsets = _c(cand_offsets, np.int64)
    req_feats = _c(req_feats)
    max_actors = 0
    if actor_ids is not None:
        actor_ids = _c(actor_ids, np.int64)
        actor_types = _c(actor_types, np.uint8)
        max_actors = int(actor_ids.shape[1])
    if doc_feats.ndim != 2 or edge_feats.ndim != 2:
        raise ValueError("doc_feats and edge_feats are 2-D")
    n_docs = int(doc_feats.shape[0])
    if author_ids.shape[0] != n_docs:
        raise ValueError("author_ids length differs from the store's row count")
    n_req = int(len(cand_offsets) - 1)
    if len(edge_offsets) != n_req + 1:
        raise ValueError("offset arrays disagree on the request count")
    total = int(cand_offsets[-1]) if n_req > 0 else 0
    out_b = out_row_bytes(doc_feats, edge_feats, req_feats, max_actors, first_degree_only)
    out_rows = np.full((total, out_b), 0xCD, dtype=np.uint8)  # poison: every byte must be written
    out_mask = np.full(total, 0xCD, dtype=np.uint8)
    rc = lib.ccr_oracle_join(
        n_docs, _ptr(doc_feats), doc_feats.shape[1] * doc_feats.dtype.itemsize, _ptr(author_ids),
        max_actors, _ptr(actor_ids), _ptr(actor_types),
        int(edge_feats.shape[1]), int(edge_feats.dtype.itemsize), int(reduce_sum_mask) & (2**64 - 1),
        n_req, _ptr(edge_keys), _ptr(edge_feats), _ptr(edge_offsets), _ptr(cand_idx), _ptr(cand_offsets),
        _ptr(req_feats), 0 if req_feats is None else req_feats.shape[1] * req_feats.dtype.itemsize,
        1 if first_degree_only else 0, _ptr(out_rows), _ptr(out_mask), int(n_threads),
    )
    if rc != 0:
        raise ValueError("the oracle does not define this case (code %d)" % rc)
    return out_rows, out_mask


def sort_edges(edge_keys: np.ndarray, edge_feats: np.ndarray, edge_offsets: np.ndarray):
    """Algorithm 1 step 1 per request: (keys, rows) in ascending key order, ties in input order.
    Returns (keys_sorted int64[E], feats_sorted like edge_feats, perm int32[E] = source index inside the request)."""
    lib = _load()
    edge_keys = _c(edge_keys, np.int64)
    edge_feats = _c(edge_feats)
    edge_offsets = _c(edge_offsets, np.int64)
    E = len(edge_keys)
    if edge_feats.shape[0] != E or int(edge_offsets[-1]) != E:
        raise ValueError("keys, rows and offsets disagree on the record count")
    keys_out = np.full(E, -0x3232323232323233, dtype=np.int64)
    feats_out = np.full(edge_feats.shape, 0, dtype=edge_feats.dtype)
    feats_out.view(np.uint8)[...] = 0xCD
    perm = np.full(E, -1, dtype=np.int32)
    row_b = int(edge_feats.shape[1] * edge_feats.dtype.itemsize)
    rc = lib.ccr_oracle_sort_edges(len(edge_offsets) - 1, _ptr(edge_keys), _ptr(edge_feats), _ptr(edge_offsets), row_b,
                                   _ptr(keys_out), _ptr(feats_out), _ptr(perm))
    if rc != 0:
        raise ValueError("malformed offsets")
    return keys_out, feats_out, perm


def resolve_ids(sorted_ids: np.ndarray, queries: np.ndarray, positions: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 6: position of each query id in the ascending id array (positions[rank] if given), or -1."""
    lib = _load()
    sorted_ids = _c(sorted_ids, np.int64)
    queries = _c(queries, np.int64)
    positions = _c(positions, np.int32)
    out = np.full(len(queries), -77, dtype=np.int32)
    lib.ccr_oracle_resolve_ids(len(sorted_ids), _ptr(sorted_ids), _ptr(positions), len(queries), _ptr(queries), _ptr(out))
    return out


def cosine_features(doc_feats, member_emb, cand_idx, cand_offsets, item_first: int, dim: int, n_chunks: int) -> np.ndarray:
    """Section 4.1.2, derived features: per-chunk cosine similarity between the request's medoid embeddings
    (member_emb float16 [n_req, n_chunks * dim]) and the candidate's item embedding (float16 elements
    [item_first, item_first + dim) of its document row), float32 arithmetic, float16 result.
    Returns uint8[C, 32]: n_chunks float16 values followed by zeros (the row's derived section, one 32-byte sector)."""
    lib = _load()
    doc_feats = _c(doc_feats)
    if doc_feats.dtype != np.float16:
        raise ValueError("the item embedding is float16")
    member_emb = _c(member_emb, np.float16)
    cand_idx = _c(cand_idx, np.int32)
    cand_offsets = _c(cand_offsets, np.int64)
    n_req = len(cand_offsets) - 1
    if member_emb.shape != (n_req, n_chunks * dim):
        raise ValueError("member_emb is [n_req, n_chunks * dim]")
    total = int(cand_offsets[-1]) if n_req > 0 else 0
    out = np.full((total, 16), 0xCDCD, dtype=np.uint16)
    rc = lib.ccr_oracle_cosine(doc_feats.shape[0], _ptr(doc_feats), doc_feats.shape[1] * 2, int(item_first), int(dim),
                               int(n_chunks), n_req, _ptr(member_emb), _ptr(cand_idx), _ptr(cand_offsets), _ptr(out))
    if rc != 0:
        raise ValueError("the oracle does not define this case (code %d)" % rc)
    return out.view(np.uint8).reshape(total, 32)


def upsert(doc_feats, author_ids, positions, new_doc_feats=None, new_author_ids=None, actor_ids=None, actor_types=None,
           new_actor_ids=None, new_actor_types=None):
    """Section 6.2, ingestion, step 3 of the per-batch protocol: batch row i is written to row positions[i] of the
    index (features and the ids stored beside them); a position outside [0, n_docs) writes nothing; an array
    for which no new values are given stays as it was.  Positions of one batch are distinct.  Returns copies
    (doc_feats, author_ids, actor_ids, actor_types)."""
    doc_feats, author_ids = np.array(doc_feats), np.array(author_ids)
    actor_ids = None if actor_ids is None else np.array(actor_ids)
    actor_types = None if actor_types is None else np.array(actor_types)
    n_docs = doc_feats.shape[0]
    seen = set()
    for i in range(len(positions)):
        p = int(positions[i])
        if p < 0 or p >= n_docs:
            continue
        if p in seen:
            raise ValueError("the oracle does not define a batch with repeated positions")
        seen.add(p)
        if new_doc_feats is not None:
            doc_feats[p] = new_doc_feats[i]
        if new_author_ids is not None:
            author_ids[p] = new_author_ids[i]
        if new_actor_ids is not None:
            actor_ids[p] = new_actor_ids[i]
        if new_actor_types is not None:
            actor_types[p] = new_actor_types[i]
    return doc_feats, author_ids, actor_ids, actor_types


def scatter_indices(cand_idx: np.ndarray, cand_offsets: np.ndarray, n_docs: int):
    """Section 6.3.1, batching and padding, step 1: from the valid-position mask (0 <= position < n_docs) the
    scatter index (batch_idx, pos_idx) of every valid candidate, pos_idx counting the request's valid
    candidates in their input order.  Returns (valid bool[C], batch_idx int64[V], pos_idx int64[V])."""
    cand_idx = np.asarray(cand_idx, dtype=np.int64)
    valid = (cand_idx >= 0) & (cand_idx < n_docs)
    batch_idx, pos_idx = [], []
    for r in range(len(cand_offsets) - 1):
        k = 0
        for j in range(int(cand_offsets[r]), int(cand_offsets[r + 1])):
            if valid[j]:
                batch_idx.append(r)
                pos_idx.append(k)
                k += 1
    return valid, np.asarray(batch_idx, dtype=np.int64), np.asarray(pos_idx, dtype=np.int64)


def join_padded(doc_feats, author_ids, edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets, n_max=None, **kw):
    """Section 6.3.1, batching and padding: T[b, n_max, row] and its mask [b, n_max].
    Step 1: scatter indices from the valid masks.  Step 2: the valid positions flattened across the batch and
    gathered in one pass (the join of `join`, per request over its valid candidates).  Step 3: scatter
    T[batch_idx, pos_idx] = gathered row.  Pads are zero rows with mask 0.  n_max defaults to max n_i.
    Returns (T uint8[b, n_max, out_b], M uint8[b, n_max], n_valid int64[b], src int64[V] flat input index of
    every kept candidate)."""
    cand_idx = np.asarray(cand_idx)
    b = len(cand_offsets) - 1
    valid, batch_idx, pos_idx = scatter_indices(cand_idx, cand_offsets, int(doc_feats.shape[0]))
    n_valid = np.bincount(batch_idx, minlength=b).astype(np.int64) if b else np.zeros(0, np.int64)
    if n_max is None:
        n_max = int(n_valid.max()) if b else 0
    flat = cand_idx[valid]                                    # step 2: flattened valid positions
    flat_offsets = np.concatenate([[0], np.cumsum(n_valid)]).astype(np.int64)
    gathered, gmask = join(doc_feats, author_ids, edge_keys, edge_feats, edge_offsets, flat, flat_offsets, **kw)
    out_b = gathered.shape[1] if gathered.ndim == 2 and gathered.shape[0] else out_row_bytes(
        doc_feats, edge_feats, kw.get("req_feats"), 0 if kw.get("actor_ids") is None else kw["actor_ids"].shape[1],
        kw.get("first_degree_only", False))
    T = np.zeros((b, n_max, out_b), dtype=np.uint8)
    M = np.zeros((b, n_max), dtype=np.uint8)
    for v in range(len(batch_idx)):                           # step 3: scatter
        if pos_idx[v] < n_max:
            T[batch_idx[v], pos_idx[v]] = gathered[v]
            M[batch_idx[v], pos_idx[v]] = gmask[v]
    return T, M, n_valid, np.nonzero(valid)[0].astype(np.int64)


def join_workload(wl, first_degree_only: bool = False, n_threads: int = 1):
    """Convenience for objects with `.store` and `.batch` attributes (duck-typed, nothing imported)."""
    s, b = wl.store, wl.batch
    return join(
        s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets,
        req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types,
        reduce_sum_mask=s.reduce_sum_mask, first_degree_only=first_degree_only, n_threads=n_threads,
    )


def half_to_float_bits(h: int) -> int:
    return int(_load().ccr_oracle_half_to_float_bits(int(h)))


def float_bits_to_half(b: int) -> int:
    return int(_load().ccr_oracle_float_bits_to_half(int(b)))
