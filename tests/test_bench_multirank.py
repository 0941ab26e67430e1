"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job aggregation, rank-0 printing."""
import json
import os
import subprocess
import sys

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)            # rank 1 is the slow one
    value = bench.whole_job_value(1000.0, world, ms)
    dist.barrier()
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_sum_of_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0                                          # max over ranks on every rank
        assert value == pytest.approx(2 * 1000.0 / 15e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert bench.whole_job_value(10.0, 1, 2.0) == pytest.approx(5000.0)


def test_reference_arm_prints_one_line_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
    r1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "1", "--workload", "config2"], env=env, capture_output=True, text=True)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env["RANK"], env["LOCAL_RANK"] = "0", "0"
    r0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "1", "--workload", "config2"], env=env, capture_output=True, text=True)
    assert r0.returncode == 0
    lines = [l for l in r0.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == d["e2e"]["unit"]
