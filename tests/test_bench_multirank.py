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


def _bench(*argv, env=None, timeout=300):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], env=env, capture_output=True,
                          text=True, timeout=timeout)


def _env_without_launcher():
    return {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`--gpus 2` with no WORLD_SIZE must not run one rank and print n_gpus 1: bench.py re-launches itself under
    torchrun (the reference arm needs no GPU, so the launcher path runs here)."""
    r = _bench("--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1", "--workload", "config2",
               "--cpu-cores", "2", env=_env_without_launcher())
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1                                         # rank 0 only
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["impl"] == "reference" and d["cpu_baseline"]["cores"] == 2


def test_gpus_flag_is_never_silently_ignored():
    import torch
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        pytest.skip("two GPUs are visible: the run would start")
    r = _bench("--gpus", "2", "--steps", "1", env=_env_without_launcher())
    assert r.returncode != 0 and "--gpus 2" in r.stderr and r.stdout.strip() == ""
    env = dict(_env_without_launcher(), WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    r = _bench("--impl", "reference", "--gpus", "2", "--steps", "1", env=env)
    assert r.returncode != 0 and "disagrees with WORLD_SIZE" in r.stderr


def test_replica_ranges_of_the_sharded_mode():
    sys.path.insert(0, ROOT)
    import bench
    assert [bench.local_replica_range(16, 4, r) for r in range(4)] == [(0, 4), (4, 4), (8, 4), (12, 4)]
    assert bench.local_replica_range(8, 1, 0) == (0, 8)
    with pytest.raises(SystemExit):
        bench.local_replica_range(8, 3, 0)
    assert bench.gather_round_losses([1.5, 2.5], 1) == [1.5, 2.5]


def _sharded_worker(rank, world, port, out):
    """One rank of the sharded mode without tensors: local loss means, a real all-gather, the controller."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from hdet_inputs import recipes as R
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import binding as B
    from paper_2604_24708_b200 import from_workload
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.config5(10)
    n = w.n_replicas
    first, n_local = bench.local_replica_range(n, world, rank)
    h = B.hdet_create(from_workload.config_for(w, n_local=n_local, replica_offset=first), [])
    B.hdet_set_schedule(h, from_workload.schedule_for(w))
    acc, n_acc, snapshots = [0.0] * n_local, 0, []
    for i in range(w.total_steps):
        perm0 = list(B.hdet_get_state(h).perm_lr[0])[:n]
        losses = R.step_losses(w, i, perm0)
        for r in range(n_local):
            acc[r] += float(losses[first + r])
        n_acc += 1
        if B.hdet_step_sharded(h, None, None):
            B.hdet_autolr_update(h, bench.gather_round_losses([x / n_acc for x in acc], world))
            acc, n_acc = [0.0] * n_local, 0
            snapshots.append(bytes(B.hdet_get_state(h)))
    st = B.hdet_get_state(h)
    out.put((rank, snapshots, [list(st.lr[g])[:n] for g in range(w.n_groups)], int(st.fired)))
    B.hdet_destroy(h)
    dist.barrier()
    dist.destroy_process_group()


def test_two_sharded_ranks_keep_byte_identical_state_for_a_whole_run():
    """Algorithm 1 over 2 gloo ranks (8 of 16 replicas each, no tensors): the round losses cross the ranks
    through a real all-gather and every rank's scalar state stays byte for byte the same, round after round;
    the rates agree with one unsharded handle fed the same losses."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_sharded_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (_, snaps0, lr0, fired0), (_, snaps1, lr1, fired1) = got
    assert len(snaps0) == 30 and snaps0 == snaps1 and fired0 == fired1 == 1
    # the same run on one unsharded handle
    sys.path.insert(0, ROOT)
    from hdet_inputs import recipes as R
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import binding as B
    from paper_2604_24708_b200 import from_workload
    w = W.config5(10)
    h = B.hdet_create(from_workload.config_for(w), [])
    B.hdet_set_schedule(h, from_workload.schedule_for(w))
    for i in range(w.total_steps):
        perm0 = list(B.hdet_get_state(h).perm_lr[0])[:w.n_replicas]
        if B.hdet_step(h, list(R.step_losses(w, i, perm0))):
            B.hdet_autolr_update(h)
    st = B.hdet_get_state(h)
    for g in range(w.n_groups):
        assert list(st.lr[g])[:w.n_replicas] == pytest.approx(lr0[g], rel=1e-13)
    B.hdet_destroy(h)
