"""Randomised GPU parity: seeded random problems x kernel-selection flags x launch tunings, each joined through
the C ABI and compared byte for byte with the CPU oracle (Eq. 1, Algorithm 1 steps 2-4).  The fixed cases of the
other test files pick the shapes that stress one path each; this one draws the combinations nobody picked."""
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


# (tile_cands, key_capacity, ws_streamers, ws_resolvers, blocks_per_sm); all zero = the defaults
TUNINGS = ((0, 0, 0, 0, 0), (256, 0, 3, 1, 0), (512, 0, 7, 7, 1), (1024, 16, 12, 4, 2), (768, 3, 2, 6, 0), (256, 200, 13, 3, 0))


def _flag_pool(B):
    return (0, B.CCR_FLAG_FORCE_GLOBAL, B.CCR_FLAG_FORCE_SAMPLED, B.CCR_FLAG_TWO_PHASE, B.CCR_FLAG_WARP_SPECIALISED,
            B.CCR_FLAG_STATIC_SPLIT, B.CCR_FLAG_WARP_SPECIALISED | B.CCR_FLAG_FORCE_GLOBAL,
            B.CCR_FLAG_TWO_PHASE | B.CCR_FLAG_FORCE_SAMPLED, B.CCR_FLAG_WARP_SPECIALISED | B.CCR_FLAG_FORCE_SAMPLED,
            B.CCR_FLAG_FORCE_SMEM, B.CCR_FLAG_TWO_PHASE | B.CCR_FLAG_FORCE_GLOBAL)


def _draw_workload(rng, it):
    second = bool(rng.integers(0, 2))
    if it % 6 == 0:  # a batch of a few thousand candidates per request, several tiles and chunks per block
        n_docs = int(rng.integers(2_000, 60_000))
        return W.config1(seed=int(rng.integers(1, 1 << 30)), n_docs=n_docs, n_req=int(rng.integers(1, 40)),
                         n_cand=int(rng.integers(100, min(9_000, n_docs // 3))), second_degree=second,
                         edge_lo=int(rng.integers(1, 50)), edge_hi=int(rng.integers(60, 9_000)))
    return tiny_workload(int(rng.integers(0, 1 << 30)), int(rng.integers(1, 300)), int(rng.integers(1, 200)),
                         int(rng.integers(0, 9)), int(rng.integers(1, 150)), int(rng.integers(1, 700)), second,
                         int(rng.choice([0, 4, 8])))


@pytest.mark.parametrize("seed", list(range(11, 23)))
def test_random_problems_flags_and_tunings(B, seed):
    rng = np.random.default_rng(seed)
    pool = _flag_pool(B)
    launches = 0
    for it in range(18):
        wl = _draw_workload(rng, it)
        if wl.batch.total_cands == 0:
            continue
        second = wl.store.actor_ids is not None
        fdo = second and bool(rng.integers(0, 2))
        want_rows, want_mask = oracle.join_workload(wl, first_degree_only=fdo, n_threads=4)
        store = B.store_from_workload(wl)
        db = B.DeviceBatch(wl.batch)
        try:
            for _ in range(4):
                flags = int(pool[int(rng.integers(0, len(pool)))]) | (B.CCR_FLAG_FIRST_DEGREE_ONLY if fdo else 0)
                tuning = TUNINGS[int(rng.integers(0, len(TUNINGS)))]
                store.set_tuning(*tuning)
                what = (seed, it, wl.name, flags, tuning, second, fdo, db.n_req, db.total_cands, db.max_edge_len)
                try:
                    rows, mask = gpu_join(store, db, flags)
                except B.CcrError as e:
                    # a forced search mode that the drawn key capacity cannot hold is refused, never degraded
                    assert e.status == B.CCR_ERR_UNSUPPORTED, what
                    continue
                launches += 1
                assert np.array_equal(mask, want_mask), what
                assert np.array_equal(rows, want_rows), what
                assert store.device_status() == B.CCR_OK, what
        finally:
            store.free()
    assert launches >= 20
