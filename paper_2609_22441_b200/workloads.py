"""Seeded synthetic inputs for the sorted-search join (store, viewers, candidate lists).

This module only *draws inputs*: it holds none of the join's arithmetic (no search, no
gather, no reduction) and is the one module shared by the CUDA path's tests/bench and by
the CPU oracle's tests.  Everything is numpy `default_rng` (PCG64) with a documented draw
order, so the same seed gives the same bytes everywhere.

Shapes follow the paper's serving workload (Section 3.1: N candidates in the tens of
thousands per request, K viewer-author affinity records in the thousands, fp16 features;
Section 6.3: a store of document features resident in GPU memory, addressed by position).
The paper measures on production traffic only, so these inputs stand in for it.

Match rate by *pool forcing*: candidate sets in production are selected because their
author (or an engager) is in the viewer's network, so most candidates do match.  A static
random store would give a match rate near K/A ~ 0.  We therefore split the docs into
`n_pools` strided pools (doc i belongs to pool i mod n_pools); viewer r owns pool r, and
`m_r` docs of that pool get their author id (and, for second-degree stores, some engager
slots) overwritten with keys of viewer r *before* the store is uploaded.

Draw order for `make_workload` (one rng, seeded once):
  1. author_ids            integers[0, A)                       int64[n_docs]
  2. doc_feats             standard_normal float32 -> dtype     [n_docs, doc_dim]   (optional)
  3. actors (if max_actors) poisson(1.5) counts clipped to max_actors, ids integers[0, A),
                           types integers[0, 3)                 int64/uint8[n_docs, max_actors]
  4. K_r for all viewers   (config specific sampler)
  5. per viewer r: keys (sorted unique sample of [0, A)), edge_feats uniform[0,1) -> fp16
  6. req_feats             standard_normal float32              [n_req, req_dim]
  7. per viewer r: forced doc choice in pool r, key choice per forced doc, (second degree:
     author coin p=.5, per-slot coins p=.6, per-slot key choice), natural candidates, shuffle
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional

import numpy as np

BASE_SEED = 260922441
ENGAGEMENT_TYPES = 3  # reacted, commented, reshared
MAX_ACTOR_SLOTS = 4


def config_seed(config: int, sub: int = 0) -> int:
    return BASE_SEED + 1000 * int(config) + int(sub)


# --------------------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------------------
@dataclass
class Store:
    """Document-feature store (one GPU = one shard), addressed by position."""

    n_docs: int
    doc_dim: int
    doc_dtype: np.dtype
    author_ids: np.ndarray  # int64[n_docs]
    doc_feats: Optional[np.ndarray]  # [n_docs, doc_dim] or None when generated elsewhere
    max_actors: int = 0
    actor_ids: Optional[np.ndarray] = None  # int64[n_docs, max_actors], empty slot = -1
    actor_types: Optional[np.ndarray] = None  # uint8[n_docs, max_actors]
    reduce_sum_mask: int = 0  # bit d set: edge dim d is summed over found engagers, else max

    @property
    def doc_row_bytes(self) -> int:
        return self.doc_dim * np.dtype(self.doc_dtype).itemsize


@dataclass
class Batch:
    """A ragged batch of requests against one store."""

    edge_dim: int
    edge_dtype: np.dtype
    req_dim: int
    req_dtype: np.dtype
    edge_keys: np.ndarray  # int64[E], ascending and unique inside each request
    edge_feats: np.ndarray  # [E, edge_dim]
    edge_offsets: np.ndarray  # int64[n_req + 1]
    cand_idx: np.ndarray  # int32[C] positions into the store
    cand_offsets: np.ndarray  # int64[n_req + 1]
    req_feats: Optional[np.ndarray]  # [n_req, req_dim] or None when req_dim == 0

    @property
    def n_req(self) -> int:
        return int(len(self.cand_offsets) - 1)

    @property
    def total_cands(self) -> int:
        return int(self.cand_offsets[-1])

    @property
    def max_edge_len(self) -> int:
        if self.n_req == 0:
            return 0
        return int(np.max(np.diff(self.edge_offsets)))

    @property
    def edge_row_bytes(self) -> int:
        return self.edge_dim * np.dtype(self.edge_dtype).itemsize

    @property
    def req_row_bytes(self) -> int:
        return self.req_dim * np.dtype(self.req_dtype).itemsize


@dataclass
class Workload:
    name: str
    seed: int
    store: Store
    batch: Batch
    meta: Dict[str, object] = field(default_factory=dict)

    def out_row_bytes(self, first_degree_only: bool = False) -> int:
        b = self.store.doc_row_bytes + self.batch.edge_row_bytes + self.batch.req_row_bytes
        if self.store.max_actors > 0 and not first_degree_only:
            b += self.batch.edge_row_bytes
        return b


def checksum64(a: Optional[np.ndarray]) -> str:
    """64-bit digest of an array's bytes (for run reports: same seed -> same digest)."""
    if a is None:
        return "none"
    return hashlib.blake2b(np.ascontiguousarray(a).view(np.uint8).reshape(-1), digest_size=8).hexdigest()


# --------------------------------------------------------------------------------------
# sampling helpers (no join arithmetic here)
# --------------------------------------------------------------------------------------
def sorted_unique_sample(rng: np.random.Generator, high: int, k: int) -> np.ndarray:
    """k distinct integers from [0, high), ascending (oversample, unique, trim)."""
    k = int(k)
    if k == 0:
        return np.empty(0, dtype=np.int64)
    if k > high:
        raise ValueError("cannot draw %d distinct values from [0, %d)" % (k, high))
    if 4 * k >= high:
        return np.sort(rng.permutation(high)[:k]).astype(np.int64)
    got = np.empty(0, dtype=np.int64)
    while len(got) < k:
        need = k - len(got)
        got = np.union1d(got, rng.integers(0, high, size=need + need // 8 + 16, dtype=np.int64))
    if len(got) > k:
        got = np.sort(got[rng.permutation(len(got))[:k]])
    return got


def distinct_sample_excluding(rng: np.random.Generator, high: int, k: int, excluded_mark: np.ndarray) -> np.ndarray:
    """k distinct integers from [0, high) whose `excluded_mark` entry is False, random order."""
    k = int(k)
    if k == 0:
        return np.empty(0, dtype=np.int64)
    got = np.empty(0, dtype=np.int64)
    rounds = 0
    while len(got) < k:
        need = k - len(got)
        draw = rng.integers(0, high, size=need + need // 4 + 16, dtype=np.int64)
        draw = draw[~excluded_mark[draw]]
        got = np.union1d(got, draw)
        rounds += 1
        if rounds == 64:  # far more rounds than a satisfiable request needs: is it satisfiable at all?
            available = int(high) - int(np.count_nonzero(excluded_mark[:high]))
            if k > available:
                raise ValueError("asked for %d distinct values but only %d are available" % (k, available))
    return got[rng.permutation(len(got))[:k]]


def zipf_clipped_lengths(lo: int, hi: int, s: float = 1.2) -> Callable[[np.random.Generator, int], np.ndarray]:
    def sample(rng: np.random.Generator, n: int) -> np.ndarray:
        return np.clip(rng.zipf(s, size=n), lo, hi).astype(np.int64)

    return sample


def log_uniform_lengths(lo: int, hi: int) -> Callable[[np.random.Generator, int], np.ndarray]:
    def sample(rng: np.random.Generator, n: int) -> np.ndarray:
        v = np.exp(rng.uniform(np.log(lo), np.log(hi), size=n))
        return np.clip(np.rint(v), lo, hi).astype(np.int64)

    return sample


def constant_lengths(k: int) -> Callable[[np.random.Generator, int], np.ndarray]:
    def sample(rng: np.random.Generator, n: int) -> np.ndarray:
        return np.full(n, int(k), dtype=np.int64)

    return sample


# --------------------------------------------------------------------------------------
# store / viewers / candidates
# --------------------------------------------------------------------------------------
def make_store(
    rng: np.random.Generator,
    n_docs: int,
    n_authors: int,
    doc_dim: int,
    doc_dtype,
    max_actors: int = 0,
    reduce_sum_mask: int = 0,
    gen_doc_feats: bool = True,
    tagged: bool = False,
) -> Store:
    author_ids = rng.integers(0, n_authors, size=n_docs, dtype=np.int64)
    doc_feats = None
    if gen_doc_feats:
        if tagged:
            # debug stores: value identifies (doc, column); exactly representable in fp32,
            # wraps harmlessly in fp16 (still a deterministic tag)
            doc_feats = (
                (np.arange(n_docs, dtype=np.int64)[:, None] * doc_dim + np.arange(doc_dim)[None, :]) % 2048
            ).astype(doc_dtype)
        else:
            doc_feats = _normal_block(rng, n_docs, doc_dim, doc_dtype)
    actor_ids = actor_types = None
    if max_actors > 0:
        counts = np.minimum(rng.poisson(1.5, size=n_docs), max_actors)
        ids = rng.integers(0, n_authors, size=(n_docs, max_actors), dtype=np.int64)
        types = rng.integers(0, ENGAGEMENT_TYPES, size=(n_docs, max_actors), dtype=np.int64).astype(np.uint8)
        slot = np.arange(max_actors)[None, :]
        used = slot < counts[:, None]
        actor_ids = np.where(used, ids, -1).astype(np.int64)
        actor_types = np.where(used, types, 0).astype(np.uint8)
    return Store(
        n_docs=int(n_docs),
        doc_dim=int(doc_dim),
        doc_dtype=np.dtype(doc_dtype),
        author_ids=author_ids,
        doc_feats=doc_feats,
        max_actors=int(max_actors),
        actor_ids=actor_ids,
        actor_types=actor_types,
        reduce_sum_mask=int(reduce_sum_mask),
    )


def _normal_block(rng: np.random.Generator, rows: int, dim: int, dtype) -> np.ndarray:
    out = np.empty((rows, dim), dtype=dtype)
    step = max(1, (1 << 22) // max(dim, 1))
    for a in range(0, rows, step):
        b = min(rows, a + step)
        out[a:b] = rng.standard_normal(size=(b - a, dim), dtype=np.float32).astype(dtype)
    return out


KEY_DISTRIBUTIONS = ("uniform", "clustered", "pareto")
KEY_OUTLIER_BASE = np.iinfo(np.int64).max - (1 << 20)  # the far outlier of a "clustered" list lies above this


def make_keys(rng: np.random.Generator, n_authors: int, k: int, key_dist: str = "uniform") -> np.ndarray:
    """k ascending unique non-negative ids.
    uniform   : a sorted unique sample of [0, n_authors) — what the benchmark configurations describe.
    clustered : member ids handed out in blocks: k - 1 consecutive ids from a random base plus one id near the top of
                the int64 range (an old or foreign account), so a linear map of the key range to buckets puts
                the whole block into one bucket.
    pareto    : heavy-tailed gaps (1 + floor of Pareto(0.5) draws scaled by 8, capped at 2^40): dense runs
                separated by a few huge jumps, so nearly every key shares a linear bucket with hundreds of others."""
    k = int(k)
    if key_dist == "uniform" or k < 2:
        return sorted_unique_sample(rng, n_authors, k)
    if key_dist == "clustered":
        base = int(rng.integers(0, max(1, n_authors - k)))
        far = KEY_OUTLIER_BASE + int(rng.integers(0, 1 << 20))
        return np.concatenate([base + np.arange(k - 1, dtype=np.int64), np.array([far], dtype=np.int64)])
    if key_dist == "pareto":
        gaps = 1 + np.minimum(np.floor(rng.pareto(0.5, size=k) * 8.0), float(1 << 40)).astype(np.int64)
        return int(rng.integers(0, max(1, n_authors))) + np.cumsum(gaps)
    raise ValueError("key_dist must be one of %s" % (KEY_DISTRIBUTIONS,))


def make_viewer(rng: np.random.Generator, n_authors: int, k: int, edge_dim: int, edge_dtype, key_dist: str = "uniform"):
    keys = make_keys(rng, n_authors, k, key_dist)
    feats = rng.random(size=(len(keys), edge_dim), dtype=np.float32).astype(edge_dtype)
    return keys, feats


def force_pool(
    rng: np.random.Generator,
    store: Store,
    keys: np.ndarray,
    pool: int,
    n_pools: int,
    m: int,
) -> np.ndarray:
    """Overwrite ids of `m` distinct docs of pool `pool` with keys of this viewer; returns the docs."""
    pool_size = (store.n_docs - pool + n_pools - 1) // n_pools if pool < store.n_docs else 0
    m = int(min(m, pool_size))
    if m <= 0 or len(keys) == 0:
        return np.empty(0, dtype=np.int64)
    docs = pool + n_pools * sorted_unique_sample(rng, pool_size, m)
    pick = keys[rng.integers(0, len(keys), size=m)]
    if store.max_actors == 0:
        store.author_ids[docs] = pick
        return docs
    has_actor = store.actor_ids[docs, 0] >= 0
    author_coin = rng.random(size=m) < 0.5
    force_author = np.where(has_actor, author_coin, True)
    store.author_ids[docs[force_author]] = pick[force_author]
    slot_coin = rng.random(size=(m, store.max_actors)) < 0.6
    slot_pick = keys[rng.integers(0, len(keys), size=(m, store.max_actors))]
    cur = store.actor_ids[docs]
    overwrite = slot_coin & (cur >= 0)
    store.actor_ids[docs] = np.where(overwrite, slot_pick, cur)
    return docs


def draw_candidates(
    rng: np.random.Generator,
    store: Store,
    forced_docs: np.ndarray,
    n_cand: int,
    n_forced: int,
    scratch_mark: np.ndarray,
) -> np.ndarray:
    """n_forced of `forced_docs` + (n_cand - n_forced) other distinct docs, shuffled; int32."""
    n_forced = int(min(n_forced, len(forced_docs), n_cand))
    if n_forced < len(forced_docs):
        take = forced_docs[rng.permutation(len(forced_docs))[:n_forced]]
    else:
        take = forced_docs
    scratch_mark[forced_docs] = True
    rest = distinct_sample_excluding(rng, store.n_docs, n_cand - n_forced, scratch_mark)
    scratch_mark[forced_docs] = False
    cand = np.concatenate([take, rest])
    rng.shuffle(cand)
    return cand.astype(np.int32)


def make_workload(
    name: str,
    seed: int,
    n_docs: int,
    n_authors: int,
    doc_dim: int,
    doc_dtype,
    edge_dim: int,
    req_dim: int,
    n_req: int,
    edge_len: Callable[[np.random.Generator, int], np.ndarray],
    n_cand,
    match: float,
    max_actors: int = 0,
    reduce_sum_mask: int = 0,
    n_pools: Optional[int] = None,
    gen_doc_feats: bool = True,
    edge_dtype=np.float16,
    req_dtype=np.float32,
    key_dist: str = "uniform",
) -> Workload:
    """One store and one ragged batch of `n_req` requests (draw order in the module docstring)."""
    rng = np.random.default_rng(seed)
    n_pools = int(n_pools or max(n_req, 1))
    store = make_store(rng, n_docs, n_authors, doc_dim, doc_dtype, max_actors, reduce_sum_mask, gen_doc_feats)
    ks = edge_len(rng, n_req)
    n_cands = np.broadcast_to(np.asarray(n_cand, dtype=np.int64), (n_req,)).copy()
    keys_l: List[np.ndarray] = []
    feats_l: List[np.ndarray] = []
    for r in range(n_req):
        k, f = make_viewer(rng, n_authors, int(ks[r]), edge_dim, edge_dtype, key_dist)
        keys_l.append(k)
        feats_l.append(f)
    req_feats = None
    if req_dim > 0:
        req_feats = rng.standard_normal(size=(n_req, req_dim), dtype=np.float32).astype(req_dtype)
    mark = np.zeros(n_docs, dtype=bool)
    cands_l: List[np.ndarray] = []
    forced_l: List[np.ndarray] = []
    # all pools are forced first, then candidates are drawn, so that a later viewer's forcing
    # cannot change an id an earlier viewer's candidate list already relies on
    for r in range(n_req):
        m = int(round(match * int(n_cands[r])))
        forced_l.append(force_pool(rng, store, keys_l[r], r % n_pools, n_pools, m))
    for r in range(n_req):
        m = int(round(match * int(n_cands[r])))
        cands_l.append(draw_candidates(rng, store, forced_l[r], int(n_cands[r]), m, mark))
    batch = assemble_batch(keys_l, feats_l, cands_l, req_feats, edge_dim, edge_dtype, req_dim, req_dtype)
    meta = {
        "n_authors": int(n_authors),
        "n_pools": n_pools,
        "match": float(match),
        "edge_len_min": int(ks.min()) if n_req else 0,
        "edge_len_max": int(ks.max()) if n_req else 0,
        "edge_len_mean": float(ks.mean()) if n_req else 0.0,
        "key_dist": key_dist,
    }
    return Workload(name=name, seed=int(seed), store=store, batch=batch, meta=meta)


def assemble_batch(keys_l, feats_l, cands_l, req_feats, edge_dim, edge_dtype, req_dim, req_dtype) -> Batch:
    n_req = len(keys_l)
    eo = np.zeros(n_req + 1, dtype=np.int64)
    co = np.zeros(n_req + 1, dtype=np.int64)
    if n_req:
        eo[1:] = np.cumsum([len(k) for k in keys_l])
        co[1:] = np.cumsum([len(c) for c in cands_l])
    edge_keys = np.concatenate(keys_l).astype(np.int64) if n_req else np.empty(0, np.int64)
    edge_feats = (
        np.concatenate(feats_l, axis=0).astype(edge_dtype) if n_req else np.empty((0, edge_dim), edge_dtype)
    )
    cand_idx = np.concatenate(cands_l).astype(np.int32) if n_req else np.empty(0, np.int32)
    return Batch(
        edge_dim=int(edge_dim),
        edge_dtype=np.dtype(edge_dtype),
        req_dim=int(req_dim),
        req_dtype=np.dtype(req_dtype),
        edge_keys=np.ascontiguousarray(edge_keys),
        edge_feats=np.ascontiguousarray(edge_feats.reshape(-1, edge_dim)),
        edge_offsets=eo,
        cand_idx=np.ascontiguousarray(cand_idx),
        cand_offsets=co,
        req_feats=None if req_feats is None else np.ascontiguousarray(req_feats),
    )


def sort_candidates_by_author(wl: Workload) -> Workload:
    """Input variant for the merge-path entry: each request's candidates stably ordered by the
    author id of the doc they point to (out-of-range positions are placed first)."""
    b, s = wl.batch, wl.store
    cand = b.cand_idx.copy()
    for r in range(b.n_req):
        lo, hi = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        seg = cand[lo:hi].astype(np.int64)
        ok = (seg >= 0) & (seg < s.n_docs)
        auth = np.where(ok, s.author_ids[np.where(ok, seg, 0)], np.iinfo(np.int64).min)
        cand[lo:hi] = seg[np.argsort(auth, kind="stable")].astype(np.int32)
    nb = Batch(**{**b.__dict__, "cand_idx": cand})
    return Workload(name=wl.name + "+sorted", seed=wl.seed, store=s, batch=nb, meta=dict(wl.meta, cands_sorted=True))


# --------------------------------------------------------------------------------------
# the five benchmark configurations (0-indexed), with size knobs for scaled-down parity cases
# --------------------------------------------------------------------------------------
SUM_DIMS_16_31 = sum(1 << d for d in range(16, 32))


def config0(seed: Optional[int] = None, n_docs: int = 100_000, n_cand: int = 20_000, k: int = 500,
            second_degree: bool = False) -> Workload:
    """Single tiny request: 100k docs x 64 fp32, A = 200k, K = 500 x 32 fp16, N = 20k, 70 % forced."""
    return make_workload(
        "config2a" if second_degree else "config0",
        config_seed(2 if second_degree else 0) if seed is None else seed,
        n_docs=n_docs, n_authors=2 * n_docs, doc_dim=64, doc_dtype=np.float32, edge_dim=32, req_dim=0,
        n_req=1, edge_len=constant_lengths(k), n_cand=n_cand, match=0.7,
        max_actors=MAX_ACTOR_SLOTS if second_degree else 0,
        reduce_sum_mask=SUM_DIMS_16_31 if second_degree else 0, n_pools=1,
    )


def config1(seed: Optional[int] = None, n_docs: int = 1_000_000, n_req: int = 64, n_cand: int = 30_000,
            second_degree: bool = False, edge_lo: int = 50, edge_hi: int = 5000, key_dist: str = "uniform") -> Workload:
    """Batched first-degree join: 1M docs x 128 fp16, A = 5M, 64 requests, K ~ clip(Zipf(1.2), 50, 5000)
    x 32 fp16, N = 30k unsorted, 16 fp32 request features; match 0.5 (limited by the pool size)."""
    return make_workload(
        "config2b" if second_degree else "config1",
        config_seed(2 if second_degree else 1, 1 if second_degree else 0) if seed is None else seed,
        n_docs=n_docs, n_authors=5 * n_docs, doc_dim=128, doc_dtype=np.float16, edge_dim=32, req_dim=16,
        n_req=n_req, edge_len=zipf_clipped_lengths(edge_lo, edge_hi, 1.2), n_cand=n_cand, match=0.5,
        max_actors=MAX_ACTOR_SLOTS if second_degree else 0,
        reduce_sum_mask=SUM_DIMS_16_31 if second_degree else 0, n_pools=n_req, key_dist=key_dist,
    )


def config3(seed: Optional[int] = None, n_docs: int = 50_000_000, n_req: int = 256, n_cand: int = 50_000,
            edge_lo: int = 10, edge_hi: int = 20_000, gen_doc_feats: bool = False,
            extra_pools: int = 160, key_dist: str = "uniform") -> Workload:
    """Production-scale store: 50M docs x 128 fp16 (+ author and engager ids), 256 requests,
    K log-uniform in [10, 20000] x 64 fp16, N = 50k, match 0.7, no request features.  The doc
    feature matrix (12.8 GB) is normally produced in chunks by `doc_feats_chunk`."""
    return make_workload(
        "config3", config_seed(3) if seed is None else seed,
        n_docs=n_docs, n_authors=n_docs, doc_dim=128, doc_dtype=np.float16, edge_dim=64, req_dim=0,
        n_req=n_req, edge_len=log_uniform_lengths(edge_lo, edge_hi), n_cand=n_cand, match=0.7,
        max_actors=MAX_ACTOR_SLOTS, reduce_sum_mask=SUM_DIMS_16_31 | (SUM_DIMS_16_31 << 32),
        n_pools=n_req + extra_pools, gen_doc_feats=gen_doc_feats, key_dist=key_dist,
    )


def doc_feats_chunk(seed: int, first: int, n: int, doc_dim: int, doc_dtype=np.float16) -> np.ndarray:
    """Rows [first, first+n) of a chunk-generated feature matrix (~N(0,1)); any chunking that
    uses multiples of DOC_CHUNK_ROWS as boundaries reproduces the same bytes."""
    if first % DOC_CHUNK_ROWS != 0:
        raise ValueError("chunks start on multiples of DOC_CHUNK_ROWS")
    out = np.empty((n, doc_dim), dtype=doc_dtype)
    for a in range(0, n, DOC_CHUNK_ROWS):
        b = min(n, a + DOC_CHUNK_ROWS)
        rng = np.random.default_rng([int(seed), (first + a) // DOC_CHUNK_ROWS, 77])
        out[a:b] = rng.standard_normal(size=(b - a, doc_dim), dtype=np.float32).astype(doc_dtype)
    return out


DOC_CHUNK_ROWS = 1 << 18


def doc_feats_chunk_device(seed: int, first: int, n: int, doc_dim: int, device):
    """Rows [first, first+n) of a production-scale feature matrix, drawn on the device (torch Philox,
    one generator seed per DOC_DEVICE_CHUNK-row block, ~N(0,1) in fp16).  Input generation only: the bytes
    it returns are what both the CUDA path and the oracle's sampled rows are taken from."""
    import torch

    if first % DOC_DEVICE_CHUNK != 0 or n > DOC_DEVICE_CHUNK:
        raise ValueError("device chunks start on multiples of DOC_DEVICE_CHUNK and hold at most that many rows")
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + first // DOC_DEVICE_CHUNK)
    return torch.randn((n, doc_dim), generator=g, device=device, dtype=torch.float32).to(torch.float16)


DOC_DEVICE_CHUNK = 1 << 22


# --- latency sweep (config 4): viewer templates on a shared store ----------------------
@dataclass
class ViewerTemplate:
    keys: np.ndarray
    feats: np.ndarray
    forced_docs: np.ndarray


def make_latency_templates(store: Store, seed: int, k_values, per_k: int, first_pool: int, n_pools: int,
                           forced_per_template: int, edge_dim: int, n_authors: int,
                           edge_dtype=np.float16) -> Dict[int, List[ViewerTemplate]]:
    """For each K in `k_values`, `per_k` viewer templates; template t owns pool first_pool + t and
    forces `forced_per_template` docs of it.  Must run before the store is uploaded."""
    rng = np.random.default_rng(seed)
    out: Dict[int, List[ViewerTemplate]] = {}
    t = 0
    for k in k_values:
        out[int(k)] = []
        for _ in range(per_k):
            keys, feats = make_viewer(rng, n_authors, int(k), edge_dim, edge_dtype)
            forced = force_pool(rng, store, keys, first_pool + t, n_pools, forced_per_template)
            out[int(k)].append(ViewerTemplate(keys, feats, forced))
            t += 1
    return out


def draw_latency_request(rng: np.random.Generator, store: Store, tpl: ViewerTemplate, n_cand: int,
                         match: float, mark: np.ndarray, edge_dim: int, edge_dtype=np.float16) -> Batch:
    cand = draw_candidates(rng, store, tpl.forced_docs, n_cand, int(round(match * n_cand)), mark)
    return assemble_batch([tpl.keys], [tpl.feats], [cand], None, edge_dim, edge_dtype, 0, np.float32)
