#!/usr/bin/env python
"""Benchmark of the batched sorted-search join on B200: `python bench.py --gpus N --steps K --warmup W`.

One step = one pass of the whole hot path (key staging, search, validate, edge/doc gather, request
broadcast, row store) over one ragged batch of synthetic requests, i.e. one `ccr_join_batch` call.
The default workload is the batched first-degree configuration (1M-doc store of 128 fp16 features, 64
requests x 30,000 candidates, Zipf(1.2) edge lists clipped to 50..5000 with 32 fp16 features, 16 fp32
request features).  Rank 0 prints ONE JSON line:

  value      candidates joined per second, whole job, inputs resident in HBM (CUDA events, max over ranks)
  e2e        the same through ccr_join_batch_host: pinned host inputs copied in, rows and mask copied out
  roofline   compulsory bytes of one launch / average launch time, against the measured HBM copy peak
  cpu_baseline  the CPU oracle as it stands, timed on this machine's host cores (rank 0, N = 1 only)

With N > 1 (torchrun, one rank per GPU) every rank joins its own batch against its own replica of the
store: the path has no exchange step, so there is no collective in the data path (weak scaling).
`--impl reference` times the CPU oracle alone on a bounded sample of the same workload.

Other workloads (`--config`): 2b second-degree; 3 / 3b / 3s production scale; 4 single-request latency sweep; and
the steps around the join — sort (Algorithm 1 step 1), resolve (Eq. 6), ingest (Section 6.2 scatter, alone and
beside the join), flow (ids -> positions -> compaction -> sort -> padded join with the cosine section, chained).
`--padded` and `--cosine` time the padded layout and the derived cosine section on the chosen workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidates_joined_per_sec"
UNIT = "candidates/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic_per_launch.txt")


def ncu_traffic(workload: str, flags: int):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel on `workload`, as recorded
    from an ncu capture in profiles/ncu_dram_traffic_per_launch.txt (columns: workload, flags, kernel, bytes per
    launch, commit the capture was taken at, summary file).  Returns (bytes, record) or (None, None) when no
    capture of that workload / flag set is on record."""
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                line = line.split("#", 1)[0].split()
                if len(line) >= 6 and line[0] == workload and int(line[1]) == int(flags):
                    return int(line[3]), {"kernel": line[2], "commit": line[4], "summary": line[5]}
    except (OSError, ValueError):
        pass
    return None, None


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=2000)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--config", default="1", choices=["1", "2b", "3", "3b", "3s", "4", "sort", "resolve", "ingest", "flow"],
                   help="1 batched first-degree (default, the headline); 2b second-degree on the same shape; 3 production-scale "
                        "store, first-degree; 3b the same on candidates sorted by author (add --flags 128 for the merge-path kernel); 3s production scale, "
                        "second-degree; 4 single-request latency sweep on the production-scale store; sort: Algorithm 1 step 1 "
                        "(per-request sort of unsorted affinity records) on the payloads of configs 1 and 3; resolve: document id -> "
                        "position over a 300M-id index (Eq. 6), batches of 1, 8 and 64 requests of 30,000 ids")
    p.add_argument("--sweep-requests", type=int, default=1000, help="requests per cell of the latency sweep")
    p.add_argument("--c3-docs", type=int, default=50_000_000, help="store size of configs 3/3b/3s (smaller for profiler captures)")
    p.add_argument("--c3-requests", type=int, default=256, help="requests of configs 3/3b/3s (smaller for profiler captures)")
    p.add_argument("--e2e-steps", type=int, default=0, help="0 = min(steps, 10)")
    p.add_argument("--flags", type=int, default=0, help="extra CCR_FLAG_* bits (experiments)")
    p.add_argument("--drop-flags", type=int, default=0, help="CCR_FLAG_* bits of the configuration to clear (experiments)")
    p.add_argument("--tile", type=int, default=0, help="candidates per ring slot (0 = library default)")
    p.add_argument("--key-cap", type=int, default=0, help="keys staged per request (0 = library default)")
    p.add_argument("--streamers", type=int, default=0)
    p.add_argument("--resolvers", type=int, default=0)
    p.add_argument("--padded", action="store_true",
                   help="time the padded batch layout: ccr_compact_valid + ccr_join_batch_padded into T[n_req, n_max]")
    p.add_argument("--cosine", action="store_true",
                   help="add the derived cosine section (3 medoids x 50 values against elements 8..57 of the document row)")
    p.add_argument("--keys", default="uniform", choices=["uniform", "clustered", "pareto"],
                   help="how the viewers' author ids are spread (configs 1 and 2b): uniform over the id range (what the benchmark "
                        "configurations describe), clustered (a block of consecutive ids plus one far outlier) or pareto "
                        "(heavy-tailed gaps)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--timed-only", action="store_true",
                   help="only warm-up and the timed region (for profiler captures): no sustain loop, e2e, latency or CPU legs")
    return p.parse_args()


def make_workload(config: str, rank: int, c3_docs: int = 50_000_000, c3_requests: int = 256, keys: str = "uniform"):
    """(workload, extra join flags) of a benchmark configuration; rank shifts the seed so replicas differ."""
    from paper_2609_22441_b200 import binding as B
    from paper_2609_22441_b200 import replicas
    from paper_2609_22441_b200 import workloads as W

    if config == "1":
        return W.config1(seed=W.config_seed(1, 0) + replicas.rank_seed_offset(rank), key_dist=keys), 0
    if config == "2b":
        return W.config1(seed=W.config_seed(2, 1) + replicas.rank_seed_offset(rank), second_degree=True, key_dist=keys), 0
    wl = W.config3(seed=W.config_seed(3, 0) + replicas.rank_seed_offset(rank), n_docs=c3_docs, n_req=c3_requests,
                   extra_pools=160 if c3_docs >= 50_000_000 else 0, key_dist=keys)
    if config == "3":
        return wl, B.CCR_FLAG_FIRST_DEGREE_ONLY
    if config == "3b":  # sorted candidates: default kernel; add --flags 128 for the merge-path kernel
        return W.sort_candidates_by_author(wl), B.CCR_FLAG_FIRST_DEGREE_ONLY | B.CCR_FLAG_CANDS_SORTED
    return wl, 0


def workload_label(wl) -> str:
    b = wl.batch
    return "%s: %d docs x %d %s, %d requests x %d candidates, edge lists %d..%d (mean %.0f) x %d fp16, %d fp32 request features" % (
        wl.name, wl.store.n_docs, wl.store.doc_dim, wl.store.doc_dtype.name, b.n_req, b.total_cands // max(b.n_req, 1),
        wl.meta["edge_len_min"], wl.meta["edge_len_max"], wl.meta["edge_len_mean"], b.edge_dim, b.req_dim)


def byte_counts(wl, mask: np.ndarray, out_b: int, second: bool):
    """Algorithmic bytes of one launch.  logical: every candidate pays for its own doc row, ids and matched
    edge rows.  compulsory: doc rows / ids once per distinct doc of the launch and edge rows once per
    distinct matched key of a request (what must cross HBM at least once); outputs are always per candidate."""
    s, b = wl.store, wl.batch
    doc_b, edge_b, req_b = s.doc_row_bytes, b.edge_row_bytes, b.req_row_bytes
    C = b.total_cands
    ids_b = 8 + (36 if second else 0)
    per_req = int(8 * len(b.edge_keys) + (req_b + 16) * b.n_req)
    found_slots = int((mask & 1).sum())
    if second:
        for sft in range(1, 5):
            found_slots += int(((mask >> sft) & 1).sum())
    logical = C * (4 + ids_b + doc_b + out_b + 1) + found_slots * edge_b + per_req
    cand = b.cand_idx.astype(np.int64)
    distinct_docs = int(len(np.unique(cand)))
    matched_keys = 0
    for r in range(b.n_req):
        c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
        hit = (mask[c0:c1] & 1).astype(bool)
        ids = [s.author_ids[cand[c0:c1][hit]]]
        if second:
            for sft in range(4):
                h = ((mask[c0:c1] >> (1 + sft)) & 1).astype(bool)
                ids.append(s.actor_ids[cand[c0:c1][h], sft])
        matched_keys += int(len(np.unique(np.concatenate(ids))))
    compulsory = C * (4 + out_b + 1) + distinct_docs * (ids_b + doc_b) + matched_keys * edge_b + per_req
    return {"logical": int(logical), "compulsory": int(compulsory), "distinct_docs": distinct_docs,
            "match_rate": float((mask & 1).mean())}


class ClockSampler:
    """nvidia-smi clock / throttle samples while the GPU is under load (one subprocess, 100 ms period)."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, mx, reasons = [], [], set()
        for t, line in self.samples:
            if t < t0 or t > t1 + 0.15:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons), "samples": len(sm)}


class NvmlClock:
    """SM clock samples straight from NVML (read-only), every few milliseconds in a thread: the latency sweep's
    cells last tens of milliseconds, too short for nvidia-smi's sampling loop."""

    def __init__(self, gpu_index: int, period_s: float = 0.005):
        self.samples = []
        self._stop = threading.Event()
        self.thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            # NVML orders devices by PCI bus id, CUDA_VISIBLE_DEVICES may remap: resolve through the CUDA device's bus id
            import torch

            bus = torch.cuda.get_device_properties(gpu_index).pci_bus_id if hasattr(
                torch.cuda.get_device_properties(gpu_index), "pci_bus_id") else None
            h = None
            if bus is not None:
                for i in range(pynvml.nvmlDeviceGetCount()):
                    hi = pynvml.nvmlDeviceGetHandleByIndex(i)
                    if pynvml.nvmlDeviceGetPciInfo(hi).bus == bus:
                        h = hi
                        break
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)

            def loop():
                while not self._stop.is_set():
                    try:
                        self.samples.append((time.time(), pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                    except Exception:
                        return
                    time.sleep(period_s)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None

    def median_mhz(self, t0: float, t1: float):
        v = [c for t, c in self.samples if t0 <= t <= t1]
        return float(np.median(v)) if v else None

    def stop(self):
        self._stop.set()


def sustain(fn, sync, t_start: float, seconds: float = 1.5):
    """Keep the measured kernels running until the loaded window is long enough for clock samples."""
    while time.time() - t_start < seconds:
        for i in range(20):
            fn(i)
        sync()


def input_checksums(wl):
    """64-bit digests of the generated inputs (same seed -> same digests on every box)."""
    from paper_2609_22441_b200 import workloads as W

    s, b = wl.store, wl.batch
    return {"author_ids": W.checksum64(s.author_ids), "doc_feats": W.checksum64(s.doc_feats) if s.doc_feats is not None else "device-generated",
            "edge_keys": W.checksum64(b.edge_keys), "edge_feats": W.checksum64(b.edge_feats), "cand_idx": W.checksum64(b.cand_idx),
            "cand_offsets": W.checksum64(b.cand_offsets)}


def config_dict(wl, bc, flags: int, args, world: int, n_buf: int = 2):
    """The `config` object of the JSON line; both arms (ours, reference) print the same one for the same run."""
    return {"workload": workload_label(wl), "l2": "inputs and outputs of a step (%.2f GB) exceed the 126 MB L2; "
            "outputs rotate over %d buffers" % (bc["compulsory"] / 1e9, n_buf),
            "match_rate": bc["match_rate"], "seed": wl.seed, "tile": args.tile or "default", "key_cap": args.key_cap or "default",
            "flags": flags, "replicas": world, "keys": args.keys}


def measured_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def time_oracle(wl, n_threads: int, repeats: int, max_cands: int = 0):
    """Seconds per pass of the CPU oracle over the first `max_cands` candidates (0 = the whole batch)."""
    from oracle import oracle
    from paper_2609_22441_b200 import workloads as W

    b = wl.batch
    if max_cands and max_cands < b.total_cands:
        co = np.minimum(b.cand_offsets, max_cands)
        b = W.Batch(**{**b.__dict__, "cand_offsets": co, "cand_idx": b.cand_idx[:max_cands]})
    s = wl.store
    best = float("inf")
    for _ in range(repeats):
        t = time.perf_counter()
        oracle.join(s.doc_feats, s.author_ids, b.edge_keys, b.edge_feats, b.edge_offsets, b.cand_idx, b.cand_offsets,
                    req_feats=b.req_feats, actor_ids=s.actor_ids, actor_types=s.actor_types,
                    reduce_sum_mask=s.reduce_sum_mask, n_threads=n_threads)
        best = min(best, time.perf_counter() - t)
    return best, int(b.total_cands)


def compact_sample(wl, kept, n_cands: int, flags: int):
    """The first n_cands candidates as a self-contained problem for the oracle: store = the rows of exactly
    those docs (kept on the host when the store was generated), candidates renumbered 0..n-1."""
    from paper_2609_22441_b200 import binding as B
    from paper_2609_22441_b200 import workloads as W

    s, b = wl.store, wl.batch
    docs = b.cand_idx[:n_cands].astype(np.int64)
    where = np.searchsorted(kept["idx"], docs)
    n_req = int(np.searchsorted(b.cand_offsets, n_cands, side="left"))
    first_only = bool(flags & B.CCR_FLAG_FIRST_DEGREE_ONLY)
    store = W.Store(n_docs=n_cands, doc_dim=s.doc_dim, doc_dtype=s.doc_dtype, author_ids=s.author_ids[docs],
                    doc_feats=kept["rows"][where], max_actors=0 if first_only else s.max_actors,
                    actor_ids=None if first_only else s.actor_ids[docs],
                    actor_types=None if first_only else s.actor_types[docs], reduce_sum_mask=s.reduce_sum_mask)
    batch = W.Batch(**{**b.__dict__, "cand_idx": np.arange(n_cands, dtype=np.int32),
                       "cand_offsets": b.cand_offsets[:n_req + 1].copy(), "edge_offsets": b.edge_offsets[:n_req + 1].copy(),
                       "req_feats": None if b.req_feats is None else b.req_feats[:n_req]})
    return W.Workload(wl.name + "-sample", wl.seed, store, batch, dict(wl.meta))


def latency_sweep(args, B, device: int):
    """Config 4: one request per launch on one stream, candidates x edge-list length grid on the
    production-scale store; p50 / p99 of the CUDA-event time and of the host time from call to stream sync."""
    import torch

    from paper_2609_22441_b200 import workloads as W

    dev = torch.device("cuda", device)
    wl = W.config3()
    s = wl.store
    n_values = (1_000, 5_000, 20_000, 50_000, 100_000)
    k_values = (10, 100, 1_000, 10_000, 20_000)
    per_k = 32
    tpl = W.make_latency_templates(s, W.config_seed(4), k_values, per_k, first_pool=256, n_pools=wl.meta["n_pools"],
                                   forced_per_template=70_000, edge_dim=wl.batch.edge_dim, n_authors=wl.meta["n_authors"])
    store, _, full = B.store_from_generated(wl, device=device, keep_all=True)  # `full`: the input matrix, for the oracle's rows
    from oracle import oracle

    oracle.build()
    cores = host_cores()
    n_oracle = 0 if args.no_cpu_baseline else min(100, args.sweep_requests)
    sampler, fine = ClockSampler(device), NvmlClock(device)
    t_sweep0 = time.time()
    oracle_cands, oracle_s = 0, 0.0
    flags = B.CCR_FLAG_FIRST_DEGREE_ONLY | args.flags
    out_b = store.out_row_bytes(flags)
    rows = torch.empty((max(n_values), out_b), dtype=torch.uint8, device=dev)
    mask = torch.empty((max(n_values),), dtype=torch.uint8, device=dev)
    mark = np.zeros(s.n_docs, dtype=bool)
    n_per_cell = args.sweep_requests
    cells = []
    launches0 = store.launch_count()
    t_all = 0.0
    c_all = 0
    for k in k_values:
        dev_tpl = [(torch.from_numpy(t.keys).to(dev), torch.from_numpy(t.feats).to(dev),
                    torch.tensor([0, len(t.keys)], dtype=torch.int64, device=dev)) for t in tpl[k]]
        for n in n_values:
            rng = np.random.default_rng(W.config_seed(4, 1000 * k_values.index(k) + n_values.index(n)))
            co = torch.tensor([0, n], dtype=torch.int64, device=dev)
            # candidate lists of the cell, pre-staged on the device
            cand = np.empty((n_per_cell, n), dtype=np.int32)
            for i in range(n_per_cell):
                t = tpl[k][i % per_k]
                n_f = min(int(round(0.7 * n)), len(t.forced_docs))
                f = t.forced_docs[rng.integers(0, len(t.forced_docs), size=n_f)] if n_f < len(t.forced_docs) else t.forced_docs
                row = np.concatenate([f[:n_f], rng.integers(0, s.n_docs, size=n - n_f)])
                rng.shuffle(row)
                cand[i] = row
            cand_dev = torch.from_numpy(cand).to(dev)
            ev, wall = [], []
            t_cell0 = None
            for i in range(-50, n_per_cell):  # 50 warm-up requests per cell
                if i == 0:
                    t_cell0 = time.time()
                j = i % n_per_cell
                keys, feats, eo = dev_tpl[j % per_k]
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize(dev)
                t0 = time.perf_counter()
                a.record()
                B.ccr_join_batch(store, 1, n, k, keys, feats, eo, cand_dev[j], co, None, rows, mask, flags)
                z.record()
                torch.cuda.synchronize(dev)
                t1 = time.perf_counter()
                if i >= 0:
                    ev.append(a.elapsed_time(z))
                    wall.append((t1 - t0) * 1e3)
            t_cell1 = time.time()
            ev.sort()
            wall.sort()
            q = lambda v, p: float(v[max(0, int(np.ceil(p * len(v))) - 1)])
            mhz = fine.median_mhz(t_cell0, t_cell1)
            cell = {"candidates": n, "edge_len": k, "event_ms_p50": q(ev, 0.5), "event_ms_p99": q(ev, 0.99),
                    "host_ms_p50": q(wall, 0.5), "host_ms_p99": q(wall, 0.99), "sm_mhz": mhz,
                    # time x clock: device cycles of the median request, comparable across runs at different clocks
                    "event_p50_kcycles": None if mhz is None else q(ev, 0.5) * mhz}
            t_all += sum(ev) * 1e-3
            c_all += n * n_per_cell
            del cand_dev
            # the oracle on the first requests of the cell, one request per call: its rows come from the generated
            # input matrix, the request becomes a compact problem (store = the request's rows) as in the parity tests
            o1, oT = [], []
            for i in range(n_oracle):
                t = tpl[k][i % per_k]
                docs = torch.from_numpy(cand[i].astype(np.int64)).to(dev)
                rows_h = full.index_select(0, docs).cpu().numpy()
                auth_h = s.author_ids[cand[i].astype(np.int64)]
                a_ = (rows_h, auth_h, t.keys, t.feats, np.array([0, len(t.keys)], np.int64), np.arange(n, dtype=np.int32),
                      np.array([0, n], np.int64))
                for threads, acc in ((1, o1), (cores, oT)):
                    t0 = time.perf_counter()
                    oracle.join(*a_, n_threads=threads)
                    acc.append((time.perf_counter() - t0) * 1e3)
                oracle_cands += n
                oracle_s += oT[-1] * 1e-3
            if o1:
                o1.sort()
                oT.sort()
                cell.update({"oracle_ms_p50_1_thread": q(o1, 0.5), "oracle_ms_p99_1_thread": q(o1, 0.99),
                             "oracle_ms_p50_all_cores": q(oT, 0.5), "oracle_ms_p99_all_cores": q(oT, 0.99)})
            cells.append(cell)
    if store.device_status() != B.CCR_OK:
        raise SystemExit("device status not clean after the sweep")
    sampler.stop()
    fine.stop()
    cpu_baseline = None
    if oracle_cands:
        cpu_baseline = {"value": oracle_cands / oracle_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": "the first %d requests of each of the 25 cells, one request per call, against a compacted copy of "
                                  "the request's document rows; per-cell p50 / p99 in latency_sweep (1 thread and all cores)" % n_oracle}
    print(json.dumps({
        "metric": METRIC, "value": c_all / t_all, "unit": UNIT, "n_gpus": 1, "steps": n_per_cell * len(cells), "warmup": 50,
        "ms_per_step": 1e3 * t_all / (n_per_cell * len(cells)), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": "config4: latency sweep, one request per launch on one stream, 50,000,000-doc store x 128 fp16, "
                   "384-byte rows, %d requests per cell (32 viewer templates per edge-list length, 70%% forced matches)" % n_per_cell,
                   "flags": flags},
        "latency_sweep": cells, "gpu_launches": int(store.launch_count() - launches0),
        "clocks": sampler.summary(t_sweep0, time.time()), "cpu_baseline": cpu_baseline,
        "input_checksums": input_checksums(wl),
        "paper_context": "the paper quotes 5-10 ms for its join on unstated Hopper-class hardware (abstract)",
    }))
    store.free()


def resolve_bench(args, B, device: int):
    """Eq. 6 on the device: b x 30,000 candidate ids resolved against a sorted array of 300M ids in HBM.
    The paper reports ~5 ms (b = 1) and ~47 ms (b = 8) for its binary-search kernel on unstated Hopper-class
    hardware, and ~1 ms for the CPU hash map it moved to."""
    import torch

    from oracle import oracle
    from paper_2609_22441_b200 import workloads as W

    dev = torch.device("cuda", device)
    n = 300_000_000
    g = torch.Generator(device=dev)
    g.manual_seed(W.config_seed(5))
    ids = torch.cumsum(torch.randint(1, 4, (n,), generator=g, device=dev, dtype=torch.int64), 0) * 2
    ix = B.IdIndex(ids, device=device)
    host = ids.cpu().numpy()
    del ids
    rng = np.random.default_rng(W.config_seed(5, 1))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    cells = []
    sampler = ClockSampler(device)
    t_leg0 = time.time()
    quick = args.timed_only  # profiler captures: the batch-64 cell alone, a handful of launches
    for b in ((64,) if quick else (1, 8, 64)):
        nq = b * 30_000
        present = host[rng.integers(0, n, size=nq)]
        q = np.where(rng.random(nq) < 0.9, present, present + 1).astype(np.int64)
        q_dev = torch.from_numpy(q).to(dev)
        out = torch.empty(nq, dtype=torch.int32, device=dev)
        for _ in range(5):
            ix.resolve(q_dev, out)
        torch.cuda.synchronize(dev)
        cold, warm = [], []
        for i in range(3 if quick else 100):
            flush.fill_(1)
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ix.resolve(q_dev, out)
            z.record()
            torch.cuda.synchronize(dev)
            cold.append(a.elapsed_time(z))
            a2, z2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a2.record()
            ix.resolve(q_dev, out)
            z2.record()
            torch.cuda.synchronize(dev)
            warm.append(a2.elapsed_time(z2))
        t_busy = time.time()
        if not quick:
            sustain(lambda i: ix.resolve(q_dev, out), lambda: torch.cuda.synchronize(dev), t_busy, 0.7)
        t0 = time.perf_counter()
        want = oracle.resolve_ids(host, q)
        t_cpu = time.perf_counter() - t0
        cold.sort()
        warm.sort()
        cells.append({"requests": b, "ids": nq, "ms_p50_L2_flushed": cold[len(cold) // 2], "ms_p99_L2_flushed": cold[min(98, len(cold) - 1)],
                      "ms_p50_repeat": warm[len(warm) // 2], "ids_per_s": nq / (cold[len(cold) // 2] * 1e-3),
                      "oracle_ms_1_core": 1e3 * t_cpu, "matches_oracle": bool(np.array_equal(out.cpu().numpy(), want)),
                      "found_fraction": float((want >= 0).mean())})
    head = cells[min(1, len(cells) - 1)]
    sampler.stop()
    print(json.dumps({
        "clocks": sampler.summary(t_leg0, time.time()),
        "cpu_baseline": {"value": head["ids"] / (head["oracle_ms_1_core"] * 1e-3), "unit": "ids/s", "cores": 1, "kind": "oracle",
                         "sample": "the headline batch (8 x 30,000 ids) once"},
        "metric": "document_ids_resolved_per_sec", "value": head["ids_per_s"], "unit": "ids/s", "n_gpus": 1, "steps": 100,
        "warmup": 5, "ms_per_step": head["ms_p50_L2_flushed"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int64", "data": "synthetic",
        "config": {"workload": "Eq. 6: ids -> positions over a sorted array of 300,000,000 ids (2.4 GB) resident in HBM; headline = "
                   "batch of 8 requests x 30,000 ids, L2 flushed between launches"},
        "cells": cells, "gpu_launches": 100,
        "paper_context": "paper: ~5 ms at batch 1, ~47 ms at batch 8 (GPU binary search, Hopper-class), ~1 ms CPU hash map",
    }))
    ix.free()


def ingest_bench(args, B, device: int):
    """Store write path (Section 6.2, ingestion step 3) and its effect on the join: a config-1 store with spare
    rows; batches of 300,000 rows (the bootstrap size, "hundreds of thousands") and of 100,000 rows (the
    steady-state size, a third of it) are scattered to new positions on an ingestion stream while the
    config-1 join runs back to back on the serving stream.  In-flight requests name live rows only, new rows go
    to positions nobody can name yet (the paper publishes ids after the write)."""
    import torch

    from paper_2609_22441_b200 import workloads as W

    dev = torch.device("cuda", device)
    wl = W.config1()
    s, b = wl.store, wl.batch
    n_live, spare = s.n_docs, 600_000
    store = B.Docstore(n_live + spare, s.doc_dim, s.doc_dtype, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype, 0, 0, device)
    store.upload(0, s.doc_feats, s.author_ids)
    db = B.DeviceBatch(b, device=device)
    C, out_b = b.total_cands, store.out_row_bytes(0)
    outs = [(torch.empty((C, out_b), dtype=torch.uint8, device=dev), torch.empty((C,), dtype=torch.uint8, device=dev))
            for _ in range(2)]
    g = torch.Generator(device=dev)
    g.manual_seed(W.config_seed(6))
    doc_t = torch.float16 if np.dtype(s.doc_dtype) == np.float16 else torch.float32
    s_join, s_ing = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    peak, peak_kind = measured_peak_gbs()

    def join(i):
        B.ccr_join_batch(store, db.n_req, C, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets, db.cand_idx,
                         db.cand_offsets, db.req_feats, outs[i % 2][0], outs[i % 2][1], 0, s_join)

    def timed(fn, n, stream):
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(n):
            fn(i)
        z.record(stream)
        return a, z

    quick = args.timed_only  # profiler captures: a handful of launches per cell
    sampler = ClockSampler(device)
    t_leg0 = time.time()
    n_join = 3 if quick else 300
    for i in range(1 if quick else 5):
        join(i)
    torch.cuda.synchronize(dev)
    a, z = timed(join, n_join, s_join)
    torch.cuda.synchronize(dev)
    join_alone_us = a.elapsed_time(z) * 1e3 / n_join
    cells = []
    for rows, order in ((300_000, "random"), (300_000, "consecutive"), (100_000, "random"), (100_000, "consecutive")):
        # several source batches (2 x 154 MB at 300k rows) so that consecutive launches do not re-read L2 lines
        srcs = []
        for k in range(2):
            pos = n_live + (torch.randperm(spare, generator=g, device=dev)[:rows] if order == "random"
                            else torch.arange(rows, device=dev) + k * rows)
            srcs.append((pos.to(torch.int32), torch.randn((rows, s.doc_dim), generator=g, device=dev, dtype=torch.float32).to(doc_t),
                         torch.randint(0, 5 * n_live, (rows,), generator=g, device=dev, dtype=torch.int64)))

        def upsert(i):
            p, d, au = srcs[i % 2]
            store.upsert(p, d, au, stream=s_ing)

        for i in range(1 if quick else 5):
            upsert(i)
        torch.cuda.synchronize(dev)
        n_up = 3 if quick else 400
        a, z = timed(upsert, n_up, s_ing)
        torch.cuda.synchronize(dev)
        up_alone_us = a.elapsed_time(z) * 1e3 / n_up
        bytes_per_batch = rows * (2 * s.doc_row_bytes + 4 + 8 + 8)
        # both at once: enough upserts queued to cover the whole join window
        n_cover = 3 if quick else int(1.3 * n_join * join_alone_us / up_alone_us) + 20
        torch.cuda.synchronize(dev)
        ua, uz = timed(upsert, n_cover, s_ing)
        ja, jz = timed(join, n_join, s_join)
        torch.cuda.synchronize(dev)
        join_busy_us = ja.elapsed_time(jz) * 1e3 / n_join
        up_busy_us = ua.elapsed_time(uz) * 1e3 / n_cover
        # the paper's regime: tens of thousands of updates per second = one steady-state batch every few seconds;
        # here one batch per 10 ms (10M rows/s at 100k rows), far above it
        cells.append({"rows_per_batch": rows, "positions": order, "upsert_alone_us": up_alone_us,
                      "upsert_alone_rows_per_s": rows / (up_alone_us * 1e-6),
                      "upsert_alone_gbs": bytes_per_batch / (up_alone_us * 1e-6) / 1e9,
                      "upsert_alone_frac_of_hbm_peak": bytes_per_batch / (up_alone_us * 1e-6) / 1e9 / peak,
                      "bytes_per_batch": bytes_per_batch,
                      "join_us_with_back_to_back_upserts": join_busy_us, "join_slowdown": join_busy_us / join_alone_us,
                      "upsert_us_with_back_to_back_joins": up_busy_us})
    if store.device_status() != B.CCR_OK:
        raise SystemExit("device status not clean")
    head = cells[0]
    sampler.stop()
    print(json.dumps({
        "clocks": sampler.summary(t_leg0, time.time()),
        "metric": "rows_upserted_per_sec", "value": head["upsert_alone_rows_per_s"], "unit": "rows/s", "n_gpus": 1, "steps": 400,
        "warmup": 5, "ms_per_step": head["upsert_alone_us"] * 1e-3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "ccr_docstore_upsert into a config-1 store (1,000,000 live rows x 256 B + 600,000 spare); batches of "
                   "300,000 / 100,000 new rows (features + author id) from device memory; join = config 1 on a second stream"},
        "roofline": {"bound": "hbm", "achieved": head["upsert_alone_gbs"], "peak": peak, "unit": "GB/s",
                     "frac": head["upsert_alone_frac_of_hbm_peak"], "traffic": None, "peak_kind": "of " + peak_kind},
        "join_alone_us": join_alone_us, "cells": cells, "gpu_launches": 400,
    }))
    store.free()


def flow_bench(args, B, device: int):
    """The whole device-side request flow on the config-1 shapes, stage by stage and chained: document ids ->
    positions (Eq. 6) -> compaction of the resolved candidates (Section 6.3.1) -> per-request sort of unsorted
    affinity records (Algorithm 1 step 1) -> join into the padded layout with the derived cosine section
    (Algorithm 1 steps 2-4, Section 4.1.2).  3 % of the candidate ids are unknown."""
    import torch

    from paper_2609_22441_b200 import workloads as W

    dev = torch.device("cuda", device)
    wl = W.config1()
    s, b = wl.store, wl.batch
    rng = np.random.default_rng(W.config_seed(7))
    doc_id = rng.permutation(10 * s.n_docs)[:s.n_docs].astype(np.int64)
    cand_ids = doc_id[b.cand_idx.astype(np.int64)]
    cand_ids = np.where(rng.random(len(cand_ids)) < 0.03, -5 - np.arange(len(cand_ids)), cand_ids)
    keys_in, feats_in = b.edge_keys.copy(), b.edge_feats.copy()
    for r in range(b.n_req):
        a, z = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
        p = rng.permutation(z - a)
        keys_in[a:z], feats_in[a:z] = b.edge_keys[a:z][p], b.edge_feats[a:z][p]
    up = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(dev)
    order = np.argsort(doc_id, kind="stable")
    store = B.store_from_workload(wl, device=device)
    store.set_cosine(8, 50, 3)
    ix = B.IdIndex(up(doc_id[order]), up(order.astype(np.int32)), device=device)
    C, n_req = len(cand_ids), b.n_req
    n_max = int(np.diff(b.cand_offsets).max())
    q, co, eo = up(cand_ids), up(b.cand_offsets), up(b.edge_offsets)
    k_in, f_in, req = up(keys_in), up(feats_in), up(b.req_feats)
    member = torch.randn((n_req, 150), device=dev).to(torch.float16)
    pos = torch.empty(C, dtype=torch.int32, device=dev)
    idx, src = torch.empty(C, dtype=torch.int32, device=dev), torch.empty(C, dtype=torch.int32, device=dev)
    offs = torch.empty(n_req + 1, dtype=torch.int64, device=dev)
    k_out, f_out = torch.empty_like(k_in), torch.empty_like(f_in)
    perm = torch.empty(len(keys_in), dtype=torch.int32, device=dev)
    flags = B.CCR_FLAG_COSINE
    out_b = store.out_row_bytes(flags)
    outs = [(torch.empty((n_req, n_max, out_b), dtype=torch.uint8, device=dev), torch.empty((n_req, n_max), dtype=torch.uint8, device=dev))
            for _ in range(2)]
    stages = {
        "resolve_ids": lambda i: ix.resolve(q, pos),
        "compact_valid": lambda i: B.ccr_compact_valid(store, n_req, C, pos, co, idx, offs, src),
        "sort_edges": lambda i: B.ccr_sort_edges(store, n_req, b.max_edge_len, k_in, f_in, eo, k_out, f_out, perm),
        "join_padded_cosine": lambda i: B.ccr_join_batch_ex(store, n_req, C, b.max_edge_len, k_out, f_out, eo, idx, offs, req,
                                                            outs[i % 2][0], outs[i % 2][1], flags, None, n_max, member),
    }

    def timed(fn, n):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize(dev)
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            fn(i)
        z.record()
        torch.cuda.synchronize(dev)
        return a.elapsed_time(z) * 1e3 / n

    n = max(20, args.steps // 10)
    sampler = ClockSampler(device)
    t_leg0 = time.time()
    for fn in stages.values():  # once in order: every stage has real inputs
        fn(0)
    per_stage = {name: timed(fn, n) for name, fn in stages.items()}

    def chain(i):
        for fn in stages.values():
            fn(i)

    chain_us = timed(chain, n)
    sustain(chain, lambda: torch.cuda.synchronize(dev), t_leg0, 1.5)
    sampler.stop()
    clocks = sampler.summary(t_leg0, time.time())
    if store.device_status() != B.CCR_OK:
        raise SystemExit("device status not clean")
    valid = int(offs[-1].item())
    print(json.dumps({
        "metric": "candidates_through_the_request_flow_per_sec", "value": C / (chain_us * 1e-6), "unit": "candidates/s",
        "n_gpus": 1, "steps": n, "warmup": 3, "ms_per_step": chain_us * 1e-3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "config-1 shapes: 64 requests x 30,000 candidate ids (3 % unknown) against a 1,000,000-id index and store; "
                   "61,823 unsorted affinity records; padded T[64, 30000, 416 B] with the cosine section; back-to-back launches, "
                   "inputs in HBM (the 15 MB of ids and the payload stay L2-warm between repetitions)"},
        "stage_us": per_stage, "chain_us": chain_us, "valid_candidates": valid, "gpu_launches": int(n), "clocks": clocks,
    }))
    ix.free()
    store.free()


def sort_bench(args, B, device: int):
    """Algorithm 1 step 1 on the device: the affinity records of every request of a batch, shuffled, are put
    back in key order by ccr_sort_edges.  Timed on the payloads of config 1 (64 lists of 50..5000 records,
    64-byte rows) and config 3 (256 lists of 10..20000 records, 128-byte rows)."""
    import torch

    from oracle import oracle
    from paper_2609_22441_b200 import workloads as W

    dev = torch.device("cuda", device)
    peak, peak_kind = measured_peak_gbs()
    results = []
    sampler = ClockSampler(device)
    t_leg0 = time.time()
    for name, wl in (("config1 payload", W.config1(n_docs=10_000, n_cand=100)),
                     ("config3 payload", W.config3(n_docs=100_000, n_cand=100, gen_doc_feats=True, extra_pools=0))):
        b = wl.batch
        rng = np.random.default_rng(wl.seed)
        keys, feats = b.edge_keys.copy(), b.edge_feats.copy()
        for r in range(b.n_req):
            a, z = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
            p = rng.permutation(z - a)
            keys[a:z], feats[a:z] = b.edge_keys[a:z][p], b.edge_feats[a:z][p]
        store = B.store_from_workload(wl, device=device)
        up = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(dev)
        k_in, f_in, eo = up(keys), up(feats), up(b.edge_offsets)
        k_out, f_out = torch.empty_like(k_in), torch.empty_like(f_in)
        p_out = torch.empty(len(keys), dtype=torch.int32, device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)  # larger than L2: written between launches
        call = lambda: B.ccr_sort_edges(store, b.n_req, b.max_edge_len, k_in, f_in, eo, k_out, f_out, p_out)
        for _ in range(3):
            call()
        torch.cuda.synchronize(dev)
        times = []
        launches0 = store.launch_count()
        for _ in range(max(args.steps // 20, 20)):
            flush.fill_(1)
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            call()
            z.record()
            torch.cuda.synchronize(dev)
            times.append(a.elapsed_time(z))
        ms = float(np.median(times))
        kernels = int(store.launch_count() - launches0)  # this library's kernels inside the timed calls of the payload
        t_busy = time.time()
        sustain(lambda i: call(), lambda: torch.cuda.synchronize(dev), t_busy, 0.8)
        E = len(keys)
        nbytes = E * (2 * (8 + b.edge_row_bytes) + 4)
        t0 = time.perf_counter()
        want = oracle.sort_edges(keys, feats, b.edge_offsets)
        t_cpu = time.perf_counter() - t0
        ok = bool(np.array_equal(k_out.cpu().numpy(), want[0]) and np.array_equal(p_out.cpu().numpy(), want[2]))
        results.append({"payload": name, "requests": b.n_req, "records": E, "longest_list": b.max_edge_len,
                        "row_bytes": b.edge_row_bytes, "ms": ms, "records_per_s": E / (ms * 1e-3),
                        "algorithmic_gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / peak,
                        "oracle_ms_1_core": 1e3 * t_cpu, "matches_oracle": ok,
                        "kernels_per_call": kernels // max(args.steps // 20, 20), "gpu_launches": kernels})
        store.free()
    head = results[-1]
    sampler.stop()
    print(json.dumps({
        "clocks": sampler.summary(t_leg0, time.time()),
        "cpu_baseline": {"value": head["records"] / (head["oracle_ms_1_core"] * 1e-3), "unit": "records/s", "cores": 1,
                         "kind": "oracle", "sample": "the config-3 payload once"},
        "metric": "edge_records_sorted_per_sec", "value": head["records_per_s"], "unit": "records/s", "n_gpus": 1,
        "steps": max(args.steps // 20, 20), "warmup": 3, "ms_per_step": head["ms"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": "Algorithm 1 step 1: per-request sort of shuffled affinity records; L2 flushed between launches",
                   "peak_kind": "of " + peak_kind},
        "roofline": {"bound": "hbm", "achieved": head["algorithmic_gbs"], "peak": peak, "unit": "GB/s",
                     "frac": head["frac_of_hbm_peak"], "traffic": None,
                     "note": "seven dependent kernels per call, each starting on flushed caches, and the shared-memory merge "
                             "sort of the chunks: latency- and instruction-bound, not by HBM"},
        "payloads": results, "gpu_launches": head["gpu_launches"],
    }))


def run_reference(args, rank: int):
    """The reference arm of this tier is the CPU oracle: rank 0 times it, the other ranks do nothing."""
    if rank != 0:
        return
    from oracle import oracle

    oracle.build()
    if args.config not in ("1", "2b"):
        print(json.dumps({"impl": "reference", "unavailable": "the CPU oracle cannot hold the 12.8 GB feature matrix of the "
                          "production-scale configurations; it is timed on configs 1 and 2b"}))
        return
    wl, cfg_flags = make_workload(args.config, 0, keys=args.keys)
    cores = host_cores()
    # one pass over the whole batch gives the mask, from which the line's config (realised match rate, bytes) is
    # written exactly as the CUDA arm writes it
    _, mask_all = oracle.join_workload(wl, n_threads=cores)
    second = wl.store.max_actors > 0
    flags = (args.flags | cfg_flags) & ~args.drop_flags
    bc = byte_counts(wl, mask_all, wl.out_row_bytes(), second)
    t_probe, n_probe = time_oracle(wl, cores, 1, max_cands=200_000)
    rate = n_probe / t_probe
    budget_s = 60.0
    sample = int(min(wl.batch.total_cands, max(30_000, rate * budget_s / max(args.steps + args.warmup, 1))))
    for _ in range(args.warmup):
        time_oracle(wl, cores, 1, max_cands=sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(wl, cores, 1, max_cands=sample)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    desc = "first %d of %d candidates of the batch per step" % (sample, wl.batch.total_cands)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": config_dict(wl, bc, flags, args, 1), "input_checksums": input_checksums(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the join has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2609_22441_b200 import binding as B
    from paper_2609_22441_b200 import build as lib_build

    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()
    B.lib()

    from paper_2609_22441_b200 import replicas

    def barrier():
        replicas.barrier(dev)

    def max_over_ranks(x: float) -> float:
        return replicas.max_over_ranks(x, dev)

    def sum_over_ranks(x: float) -> float:
        return replicas.sum_over_ranks(x, dev)

    if args.config == "4":
        if rank == 0:
            latency_sweep(args, B, local_rank)
        return
    if args.config == "resolve":
        if rank == 0:
            resolve_bench(args, B, local_rank)
        return
    if args.config == "sort":
        if rank == 0:
            sort_bench(args, B, local_rank)
        return
    if args.config == "ingest":
        if rank == 0:
            ingest_bench(args, B, local_rank)
        return
    if args.config == "flow":
        if rank == 0:
            flow_bench(args, B, local_rank)
        return
    wl, cfg_flags = make_workload(args.config, rank, args.c3_docs, args.c3_requests, args.keys)
    b = wl.batch
    second = wl.store.max_actors > 0
    kept = None
    if wl.store.doc_feats is None:
        # production-scale store: features are drawn on the device chunk by chunk; host copies are kept only
        # for the docs of the first requests, which is what the CPU baseline is timed on
        n_base = int(b.cand_offsets[min(10, b.n_req)])
        store, kept, _ = B.store_from_generated(wl, device=local_rank, keep_rows_of=b.cand_idx[:n_base])
    else:
        store = B.store_from_workload(wl, device=local_rank)
    if args.tile or args.key_cap or args.streamers or args.resolvers:
        store.set_tuning(tile_cands=args.tile, key_capacity=args.key_cap, ws_streamers=args.streamers,
                         ws_resolvers=args.resolvers)
    db = B.DeviceBatch(b, device=local_rank)
    flags = (args.flags | cfg_flags) & ~args.drop_flags
    member = None
    if args.cosine:
        store.set_cosine(8, 50, 3)
        flags |= B.CCR_FLAG_COSINE
        gm = torch.Generator(device=dev)
        gm.manual_seed(wl.seed + 7)
        member = torch.randn((db.n_req, 150), generator=gm, device=dev, dtype=torch.float32).to(torch.float16)
    out_b = store.out_row_bytes(flags)
    C = b.total_cands
    n_buf = 2  # outputs rotate so that consecutive steps do not rewrite lines still in L2
    n_out = db.n_req * db.n_max_cands if args.padded else C
    outs = [(torch.empty((n_out, out_b), dtype=torch.uint8, device=dev), torch.empty((n_out,), dtype=torch.uint8, device=dev))
            for _ in range(n_buf)]
    if args.padded:
        c_idx = torch.empty((C,), dtype=torch.int32, device=dev)
        c_src = torch.empty((C,), dtype=torch.int32, device=dev)
        c_off = torch.empty((db.n_req + 1,), dtype=torch.int64, device=dev)

    def step(i: int):
        rows, mask = outs[i % n_buf]
        if args.padded:
            B.ccr_compact_valid(store, db.n_req, C, db.cand_idx, db.cand_offsets, c_idx, c_off, c_src)
            B.ccr_join_batch_ex(store, db.n_req, C, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets, c_idx,
                                c_off, db.req_feats, rows, mask, flags, None, db.n_max_cands, member)
            return
        if args.cosine:
            B.ccr_join_batch_ex(store, db.n_req, C, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets,
                                db.cand_idx, db.cand_offsets, db.req_feats, rows, mask, flags, None, 0, member)
            return
        B.ccr_join_batch(store, db.n_req, C, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets, db.cand_idx,
                         db.cand_offsets, db.req_feats, rows, mask, flags)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    launches0 = store.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    launches = store.launch_count() - launches0
    value, ms_per_step = replicas.job_throughput(float(C), ev0.elapsed_time(ev1), args.steps, dev)
    # keep the same kernel running until the loaded window is long enough for clock samples
    while not args.timed_only and time.time() - t_wall0 < 1.2:
        for i in range(50):
            step(i)
        torch.cuda.synchronize(dev)
    t_wall1 = time.time()
    # the same steps issued alternately on two streams, as a server with two batches in flight does: the next
    # launch's blocks start on the SMs the previous launch has already left (reported beside the headline,
    # which stays the single-stream figure)
    overlapped = None
    if not args.timed_only and not args.padded and world == 1:
        streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
        torch.cuda.synchronize(dev)

        def step_on(i):
            with torch.cuda.stream(streams[i % 2]):
                step(i)

        for i in range(4):
            step_on(i)
        torch.cuda.synchronize(dev)
        o0, o1, ob = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event())
        o0.record(streams[0])
        streams[1].wait_event(o0)
        for i in range(args.steps):
            step_on(i)
        ob.record(streams[1])
        streams[0].wait_event(ob)
        o1.record(streams[0])
        torch.cuda.synchronize(dev)
        o_ms = o0.elapsed_time(o1) / args.steps
        overlapped = {"streams": 2, "ms_per_step": o_ms, "value": float(C) / (o_ms * 1e-3), "unit": UNIT}
    compact_us = None
    if args.padded:
        ev0.record()
        for i in range(200):
            B.ccr_compact_valid(store, db.n_req, C, db.cand_idx, db.cand_offsets, c_idx, c_off, c_src)
        ev1.record()
        torch.cuda.synchronize(dev)
        compact_us = ev0.elapsed_time(ev1) * 1e3 / 200
    total_cands_job = sum_over_ranks(float(C))
    if store.device_status() != B.CCR_OK:
        raise SystemExit("device status not clean after the timed region")

    # ---- end to end: pinned host inputs in, rows + mask out, through ccr_join_batch_host
    ws = B.Workspace(store, b.n_req, C, len(b.edge_keys))
    pin = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = [pin(b.edge_keys), pin(b.edge_feats.view(np.uint8)), pin(b.edge_offsets), pin(b.cand_idx), pin(b.cand_offsets),
            pin(None if b.req_feats is None else b.req_feats.view(np.uint8))]
    flags_plain = flags & ~B.CCR_FLAG_COSINE  # the host-buffer and single-request legs run without the derived section
    out_b_plain = store.out_row_bytes(flags_plain)
    h_rows = torch.empty((C, out_b_plain), dtype=torch.uint8).pin_memory()
    h_mask = torch.empty((C,), dtype=torch.uint8).pin_memory()
    h2d = int(sum(t.numel() * t.element_size() for t in h_in if t is not None))
    d2h = int(h_rows.numel() + h_mask.numel())

    def e2e_step():
        B.ccr_join_batch_host(store, ws, b.n_req, C, b.max_edge_len, len(b.edge_keys), *h_in, h_rows, h_mask, flags_plain)

    e2e_steps = args.e2e_steps or max(1, min(args.steps, 10 if C < 4_000_000 else 2))
    if args.timed_only:
        e2e_steps = 1
    for _ in range(0 if args.timed_only else 3):
        e2e_step()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1)) / e2e_steps
    e2e_value = total_cands_job / (e2e_ms * 1e-3)
    # the serving case: the rows stay on the device for the ranking model, only the mask travels back
    def e2e_step_rows_on_device():
        B.ccr_join_batch_host(store, ws, b.n_req, C, b.max_edge_len, len(b.edge_keys), *h_in, None, h_mask, flags_plain)

    for _ in range(0 if args.timed_only else 3):
        e2e_step_rows_on_device()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step_rows_on_device()
    ev1.record()
    barrier()
    e2e_dev_ms = max_over_ranks(ev0.elapsed_time(ev1)) / e2e_steps
    mask_host = h_mask.numpy().copy()
    ws.free()

    # ---- per-request latency on this batch's requests (one request per launch, device-resident inputs)
    lat = []
    if rank == 0 and not args.timed_only:
        rows0, mask0 = outs[0]
        evs = []
        for rep in range(4):
            for r in range(b.n_req):
                e0, e1 = int(b.edge_offsets[r]), int(b.edge_offsets[r + 1])
                c0, c1 = int(b.cand_offsets[r]), int(b.cand_offsets[r + 1])
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                one_eo = torch.tensor([0, e1 - e0], dtype=torch.int64, device=dev)
                one_co = torch.tensor([0, c1 - c0], dtype=torch.int64, device=dev)
                # 16-byte alignment of the key slice: start on an even key index
                e0a = e0 - (e0 & 1)
                one_eo[0] = e0 - e0a
                one_eo[1] = e1 - e0a
                if (db.edge_feats[e0a:].data_ptr() % 16) or (db.req_feats is not None and db.req_feats[r:].data_ptr() % 16):
                    continue
                torch.cuda.synchronize(dev)
                a.record()
                B.ccr_join_batch(store, 1, c1 - c0, e1 - e0a, db.edge_keys[e0a:], db.edge_feats[e0a:], one_eo,
                                 db.cand_idx[c0:], one_co, None if db.req_feats is None else db.req_feats[r:],
                                 rows0, mask0, flags_plain)
                z.record()
                evs.append((a, z))
        torch.cuda.synchronize(dev)
        lat = sorted(a.elapsed_time(z) for a, z in evs[len(evs) // 4:])

    def pct(v, q):
        return None if not v else float(v[max(0, int(np.ceil(q * len(v))) - 1)])

    if sampler is not None:
        sampler.stop()

    line = None
    if rank == 0:
        peak, peak_kind = measured_peak_gbs()
        bc = byte_counts(wl, mask_host, out_b, second and not (flags & B.CCR_FLAG_FIRST_DEGREE_ONLY))
        launch_s = ms_per_step * 1e-3  # one kernel launch per step
        achieved = bc["compulsory"] / launch_s / 1e9
        traffic, traffic_rec = (None, None) if (args.padded or args.cosine or args.keys != "uniform" or args.tile or args.key_cap) \
            else ncu_traffic(wl.name, flags)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": config_dict(wl, bc, flags, args, world, n_buf),
            "input_checksums": input_checksums(wl),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_capture": traffic_rec, "peak_kind": "of " + peak_kind,
                         "bytes_per_launch": bc["compulsory"], "logical_bytes_per_launch": bc["logical"],
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                         "logical_gbs": bc["logical"] / launch_s / 1e9},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "steps": e2e_steps},
            "e2e_rows_stay_on_device": {"value": total_cands_job / (e2e_dev_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                                        "d2h_bytes_per_step": int(h_mask.numel()), "ms_per_step": e2e_dev_ms, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "latency_ms": {"what": "one request (%d candidates) per launch, CUDA events" % (C // max(b.n_req, 1)),
                           "p50": pct(lat, 0.50), "p99": pct(lat, 0.99), "n": len(lat)},
            "clocks": sampler.summary(t_wall0, t_wall1) if sampler is not None else None,
            "two_streams": overlapped,
        }
        if args.cosine:
            line["config"]["derived"] = ("cosine section: 3 medoids x 50 values (per-request float16 member embeddings) against "
                                         "elements 8..57 of the document row, 32 more bytes per output row; e2e and latency legs "
                                         "run without it")
        if args.padded:
            line["config"]["layout"] = ("padded T[%d, %d]: a step is ccr_compact_valid (3 launches, %.1f us alone, L2-warm) + "
                                        "pad fill + join; the roofline figure divides the join's bytes by the whole step"
                                        % (db.n_req, db.n_max_cands, compact_us))
        if world == 1 and not args.no_cpu_baseline and not args.timed_only:
            from oracle import oracle

            oracle.build()
            cores = host_cores()
            if kept is None:
                t_mt, n_mt = time_oracle(wl, cores, 3)
                t_st, n_st = time_oracle(wl, 1, 1, max_cands=600_000)
                sample = "the whole batch (%d candidates), best of 3 passes" % n_mt
            else:
                sub = compact_sample(wl, kept, n_base, flags)
                t_mt, n_mt = time_oracle(sub, cores, 3)
                t_st, n_st = time_oracle(sub, 1, 1)
                sample = ("the first %d candidates (%d requests) against a compacted copy of their docs' rows, best of 3 "
                          "passes" % (n_mt, min(10, b.n_req)))
            line["cpu_baseline"] = {"value": n_mt / t_mt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": sample, "single_thread_value": n_st / t_st}
        else:
            line["cpu_baseline"] = None
    store.free()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


if __name__ == "__main__":
    main()
