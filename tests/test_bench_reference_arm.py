"""The benchmark's reference arm (`bench.py --impl reference`) runs without a GPU: it times the CPU oracle on the
headline workload and prints one JSON line with the keys the bench contract asks for."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "3"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "candidates_joined_per_sec" and line["unit"] == "candidates/s"
    assert line["n_gpus"] == 1 and line["steps"] == 1 and line["warmup"] == 3 and line["higher_is_better"] is True
    assert line["value"] > 0 and line["ms_per_step"] > 0 and line["vs_baseline"] is None and line["gpu_launches"] == 0
    # the same config keys as the CUDA arm prints for this run (workload, realised match rate, seed, flags, ...)
    cfg = line["config"]
    assert cfg["workload"].startswith("config1") and set(cfg) == {"workload", "l2", "match_rate", "seed", "tile", "key_cap", "flags", "replicas", "keys"}
    assert 0.4 < cfg["match_rate"] < 0.6 and cfg["flags"] == 0 and cfg["replicas"] == 1
    assert len(line["input_checksums"]["cand_idx"]) == 16
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and cb["sample"]
    e2e = line["e2e"]
    assert e2e["value"] == line["value"] and e2e["h2d_bytes_per_step"] == 0 and e2e["d2h_bytes_per_step"] == 0
