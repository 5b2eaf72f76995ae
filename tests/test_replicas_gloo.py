"""The N > 1 path of the benchmark on CPU: two gloo ranks, each a replica with its own workload; checks the
rank-dependent seeding and the job-level aggregation (sum of candidates / max of time)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_22441_b200 import replicas
from paper_2609_22441_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = W.config1(seed=W.config_seed(1) + replicas.rank_seed_offset(rank), n_docs=20_000, n_req=3, n_cand=400 + 100 * rank)
        local_units = float(wl.batch.total_cands)
        local_ms = 10.0 * (rank + 1)  # rank 1 is the slow one
        replicas.barrier()
        value, ms_per_step = replicas.job_throughput(local_units, local_ms, steps=5)
        mx = replicas.max_over_ranks(float(rank))
        sm = replicas.sum_over_ranks(1.0)
        out.put((rank, value, ms_per_step, mx, sm, W.checksum64(wl.batch.cand_idx), local_units))
    finally:
        dist.destroy_process_group()


def test_two_gloo_replicas_aggregate_like_the_benchmark():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, v0, ms0, mx0, sm0, ck0, u0), (r1, v1, ms1, mx1, sm1, ck1, u1) = res
    assert (r0, r1) == (0, 1)
    assert ck0 != ck1  # replicas draw different batches
    assert mx0 == mx1 == 1.0 and sm0 == sm1 == 2.0
    # every rank reports the same job-level numbers: all candidates over the slowest rank's time
    assert ms0 == ms1 == 20.0 / 5
    want = (u0 + u1) / (4.0e-3)
    assert np.isclose(v0, want) and np.isclose(v1, want)


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(3.5) == 3.5
    v, ms = replicas.job_throughput(1000.0, 50.0, steps=10)
    assert ms == 5.0 and np.isclose(v, 1000.0 / 5e-3)
