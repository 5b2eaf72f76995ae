"""TEST INFRASTRUCTURE — the naive O(N*K) scan the paper rejects (Section 3.1), kept as a pin.

For every candidate, every affinity record of the viewer is compared in turn and the first record
whose author id equals the candidate's is taken.  Pure-Python loops over numpy scalars: tiny inputs
only.  It is written independently of the C++ oracle (no search, no shared helper; fp16 handling is
numpy's own float16/float32 arithmetic), so that agreement between the two is evidence for both.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np


def _scan(keys: np.ndarray, ident: int) -> int:
    for i in range(len(keys)):
        if int(keys[i]) == ident:
            return i
    return -1


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
) -> Tuple[np.ndarray, np.ndarray]:
    n_docs = doc_feats.shape[0]
    n_req = len(cand_offsets) - 1
    second = actor_ids is not None and not first_degree_only
    rows = []
    mask = []
    for r in range(n_req):
        e0, e1 = int(edge_offsets[r]), int(edge_offsets[r + 1])
        keys = edge_keys[e0:e1]
        feats = edge_feats[e0:e1]
        zero_edge = np.zeros(edge_feats.shape[1], dtype=edge_feats.dtype)
        for j in range(int(cand_offsets[r]), int(cand_offsets[r + 1])):
            idx = int(cand_idx[j])
            m = 0
            parts = []
            if idx < 0 or idx >= n_docs:
                parts.append(np.zeros(doc_feats.shape[1], dtype=doc_feats.dtype))
                parts.append(zero_edge)
                if second:
                    parts.append(zero_edge)
            else:
                parts.append(doc_feats[idx])
                i = _scan(keys, int(author_ids[idx]))
                if i >= 0:
                    m |= 1
                    parts.append(feats[i])
                else:
                    parts.append(zero_edge)
                if second:
                    hits = []
                    for s in range(actor_ids.shape[1]):
                        act = int(actor_ids[idx, s])
                        if act < 0:
                            continue
                        i = _scan(keys, act)
                        if i >= 0:
                            hits.append(i)
                            m |= 1 << (1 + s)
                            m |= 1 << (5 + int(actor_types[idx, s]) % 3)
                    red = np.zeros(edge_feats.shape[1], dtype=np.float16)
                    for d in range(edge_feats.shape[1]):
                        if not hits:
                            continue
                        col = [feats[i][d] for i in hits]  # np.float16 scalars, slot order
                        if (reduce_sum_mask >> d) & 1:
                            acc = np.float32(0.0)
                            for v in col:
                                with np.errstate(invalid="ignore", over="ignore"):
                                    acc = np.float32(acc + np.float32(v))
                            # a NaN sum is stored as the canonical 0x7fff (the join's stated rule)
                            with np.errstate(over="ignore"):  # a finite fp32 sum above 65504 rounds to infinity
                                red[d] = np.uint16(0x7FFF).view(np.float16) if np.isnan(acc) else np.float16(acc)
                        else:
                            best = col[0]
                            for v in col[1:]:
                                if np.float32(v) > np.float32(best):
                                    best = v
                            red[d] = best
                    parts.append(red)
            if req_feats is not None:
                parts.append(req_feats[r])
            rows.append(np.concatenate([np.ascontiguousarray(p).view(np.uint8).reshape(-1) for p in parts]))
            mask.append(m)
    if rows:
        return np.stack(rows), np.asarray(mask, dtype=np.uint8)
    return np.zeros((0, 0), dtype=np.uint8), np.zeros(0, dtype=np.uint8)
