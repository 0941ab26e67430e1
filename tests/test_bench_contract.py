"""bench.py on a GPU: the JSON line carries every key of the measurement contract (small workload, few steps)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "config2", "--steps", "4",
                        "--warmup", "3", "--cpu-steps", "1", "--e2e-steps", "1", *extra],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    return json.loads(lines[0])


@pytest.mark.gpu
def test_bench_line_has_the_contract_keys():
    d = _run()
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] >= 3 and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["scaling"] == "weak" and "workload" in d["config"]
    assert d["gpu_launches"] == 4                                  # one fan-out kernel per step
    assert d["value"] == pytest.approx(8 * 25_190_400 / (d["ms_per_step"] * 1e-3), rel=1e-6)
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["frac"] == pytest.approx(r["achieved"] / r["peak"])
    assert 1000 < r["achieved"] < 9000                              # a B200 streaming kernel, not a fallback
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 8 * 25_190_400 * 2 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["unit"] == d["unit"]
    assert 1 <= c["cores"] <= c["host_cpu_count"] and f"{c['cores']} worker processes" in c["sample"]
    if c["host_cpu_count"] > 1 and len(os.sched_getaffinity(0)) > 1:
        assert c["cores"] > 1                                       # the oracle is timed on all usable host cores
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert d["device_status"] == 0


@pytest.mark.gpu
def test_bench_device_stepping_and_shared_moments_modes_run():
    d = _run("--stepping", "device", "--no-cpu-baseline", "--no-per-kernel")
    assert d["config"]["stepping"] == "device" and d["gpu_launches"] == 8    # scalar kernel + fan-out per step
    d = _run("--shared-grad", "--shared-state", "--no-cpu-baseline", "--no-per-kernel")
    assert d["roofline"]["bytes_per_element"] == pytest.approx(10.25)


@pytest.mark.gpu
def test_bench_sharded_replica_mode_runs_on_one_rank():
    """--shard-replicas with one rank: hdet_step_sharded + hdet_apply_mean (no all-reduce partner), strong-scaling units."""
    d = _run("--shard-replicas", "--sync-interval", "2", "--no-cpu-baseline")
    assert d["scaling"] == "strong" and d["n_gpus"] == 1 and d["config"]["replicas_per_gpu"] == 8
    assert d["gpu_launches"] == 4 + 2                                # four updates, two of them followed by hdet_apply_mean
    assert d["allreduce"]["rounds_timed"] == 2 and d["device_status"] == 0
    assert d["value"] == pytest.approx(8 * 25_190_400 / (d["ms_per_step"] * 1e-3), rel=1e-6)
