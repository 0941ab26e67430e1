"""Benchmark of the HDET hot path on B200: fan-out update + converge + controller call, one step per launch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config4] [--impl ours|reference] [--shard-replicas]

A step is one pass of the whole hot path over the resident workload: hdet_step (spread and schedule
scalars on the host, one fused fan-out update kernel; on the last update of a round the same kernel also
forms the replica mean) followed by hdet_autolr_update when the step ended a round.  The default
workload is the 1.3 B-parameter decoder list with N = 8 replicas and T = 1 (every step is the fused
update+converge kernel, 147 GB resident); it falls back to the 350 M list when the device has less
free memory.  Gradients are generated once on the device and held fixed during timing (147 GB of
inputs is far larger than L2, so no flush is needed).  With --gpus N > 1 every rank runs an
independent copy of the workload on its own GPU (the path has no inter-GPU exchange): weak scaling.
--shard-replicas instead splits the N replicas over the ranks, with an all-reduce of the local sums at
every round end (strong scaling).  --gpus N > 1 without a launcher starts the N ranks itself.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from hdet_inputs import recipes as R  # noqa: E402
from hdet_inputs import workloads as W  # noqa: E402

METRIC = "fan-out step+converge throughput (replica-parameter-elements updated per second)"
UNIT = "replica-param-elements/s"
# DRAM bytes per replica-element of fanout_kernel<bf16, AdamW, converge> (the bulk-copy kernel), from the ncu capture
# of that kernel on the 25 M list summarised under profiles/ (5.1818 GB over 8 x 25,190,400 elements); traffic grows
# in proportion to N x P.  Set to None whenever that kernel changes until the counters are taken again.
NCU_DRAM_BYTES_PER_ELEMENT_ADAMW_BF16_CONVERGE = 5.1818e9 / (8 * 25_190_400)
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


def bytes_per_element(w: W.Workload, shared_grad: bool = False, shared_state: bool = False, bf16_copy: bool = False) -> float:
    """Algorithmic HBM bytes per replica-parameter-element of the fan-out kernel (fused converge adds none).

    A shared gradient is read once per N replicas; shared moments are read and written once per N replicas.
    The gradient replica-mean mode reads every replica's gradient, like the per-replica mode.
    """
    n = w.n_replicas
    g = (2 if w.grad_dtype == W.DTYPE_BF16 else 4) / (n if shared_grad else 1)
    if bf16_copy:                                    # 2 bytes per PARAMETER at every converge, i.e. every T steps
        g += 2 / (n * w.sync_interval)
    if w.optimizer == W.OPT_ADAMW:
        state = 16 / (n if shared_state else 1)      # m, v read and written
        return 8 + g + state                         # theta read and written
    return 8 + g + (8 if w.momentum else 0)          # SGD; the momentum buffer is read and written


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def oracle_sample(w: W.Workload, n_slabs: int, slab: int = 65536):
    """Bounded sample of the workload for the CPU oracle: n_slabs ranges of `slab` elements from the largest tensors."""
    big = sorted(range(len(w.tensors)), key=lambda k: -w.tensors[k].numel)
    slabs = []
    for j in range(n_slabs):
        k = big[j % max(1, min(len(big), 8))]
        n = min(slab, w.tensors[k].numel)
        start = (j * 7919 * slab) % max(1, w.tensors[k].numel - n + 1)
        slabs.append((k, start // 8 * 8, n))
    return slabs


class OracleBench:
    """The CPU oracle, as it stands, on a bounded sample, one worker process per usable host core.

    Every worker holds its own share of the sample (8 ranges of 65,536 elements x N replicas) and runs the
    oracle's step on it with the gradients held fixed, as on the GPU; all workers run at the same time and the
    wall time of the slowest counts.  The worker processes are started with `spawn` (a process forked after the
    first CUDA call would hang).
    """
    SLABS_PER_WORKER = 8

    def __init__(self, w: W.Workload, cores=None):
        from oracle import driver as OD                      # test infrastructure: only this leg may use it
        self.w = w
        self.cores = cores or OD.usable_cores()
        self.slabs = oracle_sample(w, self.SLABS_PER_WORKER * self.cores)
        self.pool = OD.OraclePool(w, self.slabs, n_workers=self.cores)
        self.cores = self.pool.n_workers
        self.units = sum(n for (_, _, n) in self.slabs) * w.n_replicas

    def time_steps(self, steps: int) -> float:
        return self.pool.time_steps(steps)

    def close(self):
        self.pool.close()

    def describe(self):
        return (f"{len(self.slabs)} ranges x {self.slabs[0][2]} elements x N={self.w.n_replicas} replicas of "
                f"{self.w.name} ({self.units} replica-elements per step) split over {self.cores} worker processes, "
                f"gradients held fixed")


def time_oracle(w, steps, warmup, cores=None):
    """(bench object, replica-elements per second over all workers, seconds per step)."""
    ob = OracleBench(w, cores)
    try:
        if warmup:
            ob.time_steps(warmup)
        dt = ob.time_steps(steps)
    finally:
        ob.close()
    return ob, ob.units * steps / dt, dt / steps


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu = gpu_index
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            for nm, val in zip(names, p[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = sm[len(sm) // 4:] if len(sm) >= 4 else sm      # skip the ramp at the start
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(ms: float, world: int, device="cpu") -> float:
    """The slowest rank's time: every multi-GPU number is the max over ranks, never a mean or a wall clock."""
    if world == 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Units all ranks processed per second (each rank runs its own copy of the job: weak scaling)."""
    return units_per_rank * world / (ms_per_step * 1e-3)


def pick_workload(name, torch, sync_interval=None, optimizer=None, grad_dtype=None):
    """The named workload, optionally with another T, optimizer or gradient type (same tensor list and inputs)."""
    from dataclasses import replace
    w = W.ALL_CONFIGS[name]()
    if sync_interval:
        w = replace(w, sync_interval=sync_interval, name=f"{w.name}_T{sync_interval}")
    if optimizer == "sgd":
        w = replace(w, optimizer=W.OPT_SGD, momentum=0.0, name=f"{w.name}_sgd")
    elif optimizer == "sgd-momentum":
        w = replace(w, optimizer=W.OPT_SGD, momentum=0.9, name=f"{w.name}_sgd_momentum")
    elif optimizer == "adamw":
        w = replace(w, optimizer=W.OPT_ADAMW, momentum=0.0, name=f"{w.name}_adamw")
    if grad_dtype:
        w = replace(w, grad_dtype=W.DTYPE_F32 if grad_dtype == "f32" else W.DTYPE_BF16, name=f"{w.name}_g{grad_dtype}")
    gsz = 2 if w.grad_dtype == W.DTYPE_BF16 else 4
    state = 8 if w.optimizer == W.OPT_ADAMW else (4 if w.momentum else 0)
    need = w.n_replicas * w.arena_numel() * (4 + gsz + state)
    free, _ = torch.cuda.mem_get_info()
    note = None
    if need + (3 << 30) > free:
        note = f"{name} needs {need / 1e9:.1f} GB but only {free / 1e9:.1f} GB are free: fell back to config3"
        w = W.config3()
    return w, note


def run_ours(args):
    import torch
    import torch.distributed as dist

    from hdet_inputs import device as D
    from paper_2604_24708_b200 import binding as B
    from paper_2604_24708_b200 import from_workload
    from paper_2604_24708_b200.arena import StackedArena

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))

    w, note = pick_workload(args.workload, torch, args.sync_interval, args.optimizer, args.grad_dtype)
    n, P = w.n_replicas, w.numel
    arena = StackedArena([t.numel for t in w.tensors], [t.group for t in w.tensors], n, w.optimizer, w.grad_dtype,
                         device=f"cuda:{local}", align_elems=w.align_elems, shared_grad=args.shared_grad,
                         shared_state=args.shared_state, sgd_momentum=(w.optimizer == W.OPT_SGD and w.momentum != 0.0),
                         bf16_copy=args.bf16_copy)
    D.fill(arena.param[0], R.param_key(w), 0, R.param_scale(w))
    for r in range(1, n):
        arena.param[r].copy_(arena.param[0])
    if args.shared_grad:
        D.fill(arena.grad, R.grad_key(w, 0, 0), 0, R.grad_scale(w))
    else:
        for r in range(n):
            D.fill(arena.grad[r], R.grad_key(w, 0, r), 0, R.grad_scale(w))
    grad_mode = B.HDET_GRAD_REPLICA_MEAN if args.grad_mode == "mean" else B.HDET_GRAD_AS_GIVEN
    h = B.hdet_create(from_workload.config_for(w, fuse=1, device=local, grad_mode=grad_mode), arena.descriptors())
    B.hdet_set_schedule(h, from_workload.schedule_for(w))
    stream = torch.cuda.current_stream()
    losses = [list(R.step_losses(w, i % w.total_steps)) for i in range(w.total_steps)]
    state = {"i": 0}

    d_losses = torch.tensor(np.array(losses), dtype=torch.float64, device=f"cuda:{local}")
    steps_per_call = 1
    graph = None

    def one_step():
        """One update (or, with --stepping graph, one recorded round of T updates)."""
        k = state["i"] % w.total_steps
        if args.stepping == "host":
            if B.hdet_step(h, losses[k], stream.cuda_stream):
                B.hdet_autolr_update(h)
        elif args.stepping == "device":
            B.hdet_step_device(h, d_losses[k], stream.cuda_stream)
        else:
            graph.replay()
        state["i"] += steps_per_call

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.stepping == "graph":
        # One round of T device-resident updates is run directly (uploads the state), then recorded once;
        # every call of one_step() replays the recorded round.
        T = w.sync_interval
        if args.steps % T:
            raise SystemExit(f"--stepping graph needs --steps to be a multiple of the sync interval {T}")
        for k in range(T):
            B.hdet_step_device(h, d_losses[k % w.total_steps], stream.cuda_stream)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        before = B.hdet_kernel_launches(h)
        with torch.cuda.graph(graph, stream=side):
            for k in range(T):
                B.hdet_step_device(h, d_losses[k % w.total_steps], torch.cuda.current_stream().cuda_stream)
        launches_per_call = B.hdet_kernel_launches(h) - before
        steps_per_call = T
    n_calls = args.steps // steps_per_call
    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()

    # ---- device-timed region: inputs resident in HBM -------------------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = B.hdet_kernel_launches(h)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_calls + 1)]
    barrier()
    ev[0].record(stream)
    for k in range(n_calls):
        one_step()
        ev[k + 1].record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    launches = B.hdet_kernel_launches(h) - launches0
    if args.stepping == "graph":
        launches = launches_per_call * n_calls          # replays launch the recorded kernels without calling the library
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step_ms = [ev[k].elapsed_time(ev[k + 1]) / steps_per_call for k in range(n_calls)]
    ms_per_step = max_over_ranks(total_ms, world, f"cuda:{local}") / args.steps
    value = whole_job_value(n * P, world, ms_per_step)

    # ---- end-to-end region: this step's gradients come from pinned host memory, the status word goes back --
    n_grad_copies = 1 if args.shared_grad else n
    h2d_bytes = n_grad_copies * arena.p_pad * arena.grad.element_size()
    # ten steps where a step's upload is small; three where one step already moves gigabytes over PCIe
    e2e_steps = args.e2e_steps if args.e2e_steps else (3 if h2d_bytes > (4 << 30) else 10)
    e2e_steps = max(1, e2e_steps)
    # Host stepping goes through hdet_step_host_grads: the library itself copies every tensor's gradients from a
    # pinned host image of the gradient arena (same layout as on the device) and then launches the update.
    host_image, host_ptrs, host_grad = None, None, None
    if args.stepping == "host" and h2d_bytes <= (48 << 30):
        try:
            host_image = torch.empty(arena.grad.shape, dtype=arena.grad.dtype).pin_memory()
            host_image.copy_(arena.grad)
            gsz = arena.grad.element_size()
            host_ptrs = [host_image.data_ptr() + gsz * off for off in arena.offsets]
        except RuntimeError:
            host_image = None
    if host_image is None:
        host_grad = torch.empty(arena.p_pad, dtype=arena.grad.dtype).pin_memory()
        host_grad.copy_((arena.grad if args.shared_grad else arena.grad[0]).cpu())

    def e2e_step():
        k = state["i"] % w.total_steps
        if host_image is not None:
            if B.hdet_step_host_grads(h, host_ptrs, losses[k], stream.cuda_stream):
                B.hdet_autolr_update(h)
            state["i"] += 1
        else:
            for r in range(n_grad_copies):
                (arena.grad if args.shared_grad else arena.grad[r]).copy_(host_grad, non_blocking=True)
            if args.stepping == "host":
                one_step()
            else:                                           # per step, so that every step sees its own gradients
                B.hdet_step_device(h, d_losses[k], stream.cuda_stream)
                state["i"] += 1
        st = B.hdet_get_state(h, raise_on_nonfinite=False)   # reads the device status word back (synchronises)
        return st.device_status

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, f"cuda:{local}")
    e2e_value = whole_job_value(n * P, world, e2e_ms / e2e_steps)
    final_state = B.hdet_get_state(h, raise_on_nonfinite=False)
    B.hdet_destroy(h)

    # ---- each kernel of the path on its own (same arena, a few launches each, after the headline timing) ----
    per_kernel = {}
    if not args.no_per_kernel:
        from dataclasses import replace as _replace

        def timed(fn, reps=5):
            fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        bpe_step = bytes_per_element(_replace(w, sync_interval=1 << 40), args.shared_grad, args.shared_state)
        for label, T, fuse, bpe_k in (("fanout_update", 1 << 40, 1, bpe_step),
                                      ("fanout_update_converge_fused", 1, 1, bpe_step),
                                      ("fanout_update_then_converge_unfused", 1, 0, bpe_step + 8)):
            wk = _replace(w, sync_interval=T, autolr=0)
            hk = B.hdet_create(from_workload.config_for(wk, fuse=fuse, device=local, grad_mode=grad_mode), arena.descriptors())
            B.hdet_set_schedule(hk, from_workload.schedule_for(wk))
            ms = timed(lambda: B.hdet_step(hk, None, stream.cuda_stream))
            per_kernel[label] = {"ms": ms, "GB_per_s": bpe_k * n * P / ms / 1e6, "bytes_per_element": bpe_k}
            if label == "fanout_update":
                ms = timed(lambda: B.hdet_converge(hk, stream.cuda_stream))
                per_kernel["converge_standalone"] = {"ms": ms, "GB_per_s": 8 * n * P / ms / 1e6, "bytes_per_element": 8}
            if label == "fanout_update":
                # Eq. 10 (three kernels): reads the checkpoint twice (norm, then fan-out) and writes all N replicas
                ms = timed(lambda: B.hdet_warm_init(hk, 0.01, 1, stream.cuda_stream), reps=3)
                wb = (8 + 4 * n) * P
                per_kernel["warm_init"] = {"ms": ms, "GB_per_s": wb / ms / 1e6, "bytes_per_element": wb / (n * P)}
            B.hdet_destroy(hk)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    bpe = bytes_per_element(w, args.shared_grad, args.shared_state, args.bf16_copy)
    peak, peak_src = measured_peaks()
    # mean duration of one fan-out launch: a step is one fan-out launch (device stepping adds one-warp scalar kernels)
    launch_ms = statistics.mean(per_step_ms)
    achieved = bpe * n * P / (launch_ms * 1e-3) / 1e9
    traffic, traffic_src = args.traffic_bytes, "command line" if args.traffic_bytes else None
    plain_mode = not (args.shared_grad or args.shared_state or args.grad_mode == "mean" or args.bf16_copy)
    if (traffic is None and plain_mode and NCU_DRAM_BYTES_PER_ELEMENT_ADAMW_BF16_CONVERGE and w.optimizer == W.OPT_ADAMW
            and w.grad_dtype == W.DTYPE_BF16 and w.sync_interval == 1):
        traffic = NCU_DRAM_BYTES_PER_ELEMENT_ADAMW_BF16_CONVERGE * n * P
        traffic_src = "ncu dram__bytes_read+write on the 25 M list, scaled by N*P (see profiles/)"
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (bf16 gradients, fp64 replica sum)" if w.grad_dtype == W.DTYPE_BF16 else "f32",
        "data": "synthetic (seeded integer generator; gradients held fixed during timing)",
        "config": {
            "workload": w.name, "n_replicas": n, "params_per_replica": P, "n_tensors": len(w.tensors),
            "optimizer": "adamw" if w.optimizer == W.OPT_ADAMW else "sgd", "sync_interval": w.sync_interval,
            "alpha_lr": w.alpha_lr, "stepping": args.stepping, "grad_mode": args.grad_mode, "shared_grad": args.shared_grad,
            "shared_moments": args.shared_state, "bf16_copy": args.bf16_copy, "resident_gb": arena.resident_bytes() / 1e9,
            "l2_policy": "inputs larger than L2 (no flush)", "parallelism": f"{world} independent replicas of the job",
            "note": note,
        },
        "param_elements_per_s": value / n,
        "hbm_frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": 4,
                "steps": e2e_steps,
                "what": ("per step: hdet_step_host_grads copies the gradients of all replicas from pinned host memory "
                         "and updates (+ hdet_autolr_update); device status word read back") if host_image is not None
                else "per step: gradients copied from pinned host memory by the caller, then the step; status word read back"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_src,
                     "kernel": ("fanout_shared_kernel" if args.shared_state else "fanout_kernel") + (" (fused update+converge)" if w.sync_interval == 1 else ""),
                     "bytes_per_element": bpe, "launch_ms": launch_ms},
        "per_kernel": per_kernel,
        "device_status": int(final_state.device_status),
    }
    if world == 1 and not args.no_cpu_baseline:
        ob, v, sec = time_oracle(w, args.cpu_steps, 1, args.cpu_cores)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": ob.cores, "host_cpu_count": os.cpu_count(),
                               "kind": "oracle", "sample": ob.describe(), "s_per_step": sec, "steps": args.cpu_steps}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def gather_round_losses(local_means, world: int, device="cpu"):
    """Algorithm 1's all-gather of the per-replica round losses: every rank contributes the means of its local
    replicas and receives all N, in replica order (ranks hold consecutive replicas)."""
    if world == 1:
        return [float(x) for x in local_means]
    import torch
    import torch.distributed as dist
    mine = torch.tensor(list(local_means), dtype=torch.float64, device=device)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    return [float(x) for p in parts for x in p.cpu()]


def local_replica_range(n_replicas: int, world: int, rank: int):
    """Replicas [first, first + count) held by `rank` when N replicas are split evenly over `world` ranks."""
    if n_replicas % world:
        raise SystemExit(f"--shard-replicas needs the replica count {n_replicas} to be a multiple of the {world} ranks")
    count = n_replicas // world
    return rank * count, count


def run_sharded(args):
    """Replica axis sharded over the ranks (the paper's own arrangement): every rank holds N / world replicas.

    Per step hdet_step_sharded; at a round end the fused kernel leaves the sums over the local replicas in a
    staging buffer, the ranks all-reduce it (the one exchange of Eq. 3, P floats), hdet_apply_mean writes
    sum / N to the local replicas, the round losses are all-gathered (N doubles) and hdet_autolr_update runs
    the controller on every rank.  Total work is fixed as ranks are added: strong scaling.
    """
    import torch
    import torch.distributed as dist

    from hdet_inputs import device as D
    from paper_2604_24708_b200 import binding as B
    from paper_2604_24708_b200 import from_workload
    from paper_2604_24708_b200.arena import StackedArena

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    w, note = pick_workload(args.workload, torch, args.sync_interval)
    n, P = w.n_replicas, w.numel
    first, n_local = local_replica_range(n, world, rank)
    arena = StackedArena([t.numel for t in w.tensors], [t.group for t in w.tensors], n_local, w.optimizer, w.grad_dtype,
                         device=dev, align_elems=w.align_elems)
    D.fill(arena.param[0], R.param_key(w), 0, R.param_scale(w))
    for r in range(1, n_local):
        arena.param[r].copy_(arena.param[0])
    for r in range(n_local):                                  # local replica r is global replica first + r
        D.fill(arena.grad[r], R.grad_key(w, 0, first + r), 0, R.grad_scale(w))
    h = B.hdet_create(from_workload.config_for(w, fuse=1, device=local, n_local=n_local, replica_offset=first),
                      arena.descriptors())
    B.hdet_set_schedule(h, from_workload.schedule_for(w))
    _, total = B.hdet_partial_layout(h, len(w.tensors))
    partial = torch.zeros(total, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    acc = [0.0] * n_local
    state = {"i": 0, "n_acc": 0, "rounds": 0}
    ar_events = []

    def one_step(timed=False):
        i = state["i"]
        perm0 = list(B.hdet_get_state(h).perm_lr[0])[:n]
        losses = R.step_losses(w, i % w.total_steps, perm0)
        for r in range(n_local):
            acc[r] += float(losses[first + r])
        state["n_acc"] += 1
        if B.hdet_step_sharded(h, None, partial, stream.cuda_stream):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            if world > 1:
                dist.all_reduce(partial)                       # on the current (= launch) stream's order
            b.record(stream)
            if timed:
                ar_events.append((a, b))
            B.hdet_apply_mean(h, partial, stream.cuda_stream)
            means = [x / state["n_acc"] for x in acc]
            B.hdet_autolr_update(h, gather_round_losses(means, world, dev))
            for r in range(n_local):
                acc[r] = 0.0
            state["n_acc"] = 0
            state["rounds"] += 1
        state["i"] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = B.hdet_kernel_launches(h)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        one_step(timed=True)
    e1.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    launches = B.hdet_kernel_launches(h) - launches0
    ms_per_step = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    ar_ms = sum(a.elapsed_time(b) for a, b in ar_events)
    ar_ms = max_over_ranks(ar_ms, world, dev)
    final_state = B.hdet_get_state(h, raise_on_nonfinite=False)
    B.hdet_destroy(h)
    if rank == 0:
        value = n * P / (ms_per_step * 1e-3)                   # all N replicas of the one job, whatever the rank count
        bpe = bytes_per_element(w)
        peak, peak_src = measured_peaks()
        rounds = max(1, len(ar_events))
        # per GPU and step: the local update (26 B per local replica-element); per round end additionally the
        # staging buffer written (4 B per parameter), read and the mean written to the local replicas
        local_bytes = bpe * n_local * P
        achieved = local_bytes * world / (ms_per_step * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32 (bf16 gradients, fp64 replica sum)" if w.grad_dtype == W.DTYPE_BF16 else "f32",
            "data": "synthetic (seeded integer generator; gradients held fixed during timing)",
            "config": {"workload": w.name, "n_replicas": n, "replicas_per_gpu": n_local, "params_per_replica": P,
                       "sync_interval": w.sync_interval, "l2_policy": "inputs larger than L2 (no flush)",
                       "parallelism": f"replica axis sharded over {world} GPU(s): hdet_step_sharded, all-reduce of "
                                      f"{total} fp32 sums per round, hdet_apply_mean", "note": note},
            "gpu_launches": int(launches), "clocks": clocks,
            "allreduce": {"rounds_timed": len(ar_events), "ms_per_round": ar_ms / rounds,
                          "share_of_step_time": ar_ms / (ms_per_step * args.steps), "bytes_per_round": 4 * total},
            "roofline": {"bound": "hbm", "achieved": achieved / world, "peak": peak, "unit": "GB/s",
                         "frac": achieved / world / peak, "traffic": None, "peak_source": peak_src,
                         "kernel": "fanout_kernel (per GPU; algorithmic bytes of the update only)",
                         "bytes_per_element": bpe},
            "e2e": None, "device_status": int(final_state.device_status),
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def relaunch_under_torchrun(args):
    """`--gpus N` without a launcher: start the N ranks here (what the driver's torchrun line does)."""
    import socket
    if args.impl == "ours":
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: only {have} CUDA device(s) visible; "
                             f"nothing was run (a smaller run would misreport n_gpus)")
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.run(cmd).returncode)


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample per step (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = W.ALL_CONFIGS[args.workload]()
    ob, v, sec = time_oracle(w, args.steps, max(args.warmup, 1), args.cpu_cores)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    out = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded integer generator)",
        "config": {"workload": w.name, "n_replicas": w.n_replicas, "params_per_replica": w.numel,
                   "sample": ob.describe()},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": ob.cores, "host_cpu_count": os.cpu_count(), "kind": "oracle",
                         "sample": ob.describe()},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config4", choices=sorted(W.ALL_CONFIGS))
    ap.add_argument("--sync-interval", type=int, default=None,
                    help="override the workload's T (e.g. 1 to profile the fused update+converge kernel on a small list)")
    ap.add_argument("--stepping", default="host", choices=["host", "device", "graph"],
                    help="host: hdet_step (+ hdet_autolr_update); device: hdet_step_device with device losses; "
                         "graph: a recorded round of hdet_step_device calls replayed")
    ap.add_argument("--grad-mode", default="as_given", choices=["as_given", "mean"],
                    help="mean: every replica steps with the on-device replica mean of the gradients")
    ap.add_argument("--shared-grad", action="store_true", help="one gradient for all replicas (grad_stride 0)")
    ap.add_argument("--shared-state", action="store_true",
                    help="one pair of Adam moments for all replicas (needs --shared-grad or --grad-mode mean)")
    ap.add_argument("--optimizer", default=None, choices=["adamw", "sgd", "sgd-momentum"],
                    help="run the workload's tensor list with another optimizer (sgd: Eq. 2; sgd-momentum: mu = 0.9)")
    ap.add_argument("--grad-dtype", default=None, choices=["bf16", "f32"], help="override the workload's gradient type")
    ap.add_argument("--bf16-copy", action="store_true",
                    help="every converge also writes the averaged parameters as bf16 (hdet_tensor.param_bf16)")
    ap.add_argument("--e2e-steps", type=int, default=0,
                    help="steps of the end-to-end region (default: 10, or 3 when one step uploads more than 4 GB)")
    ap.add_argument("--cpu-steps", type=int, default=30)
    ap.add_argument("--cpu-cores", type=int, default=None,
                    help="worker processes of the CPU oracle (default: every core this process may use)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-kernel", action="store_true", help="skip the per-kernel timings that follow the headline run")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="dram bytes per launch of the dominant kernel from an ncu capture (reported as roofline.traffic)")
    ap.add_argument("--shard-replicas", action="store_true",
                    help="split the replica axis over the ranks (N / world replicas per GPU, all-reduce of the local "
                         "sums at every round end) instead of running one independent copy of the job per GPU")
    args = ap.parse_args()
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        relaunch_under_torchrun(args)
    if world_env is not None and int(world_env) != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} disagrees with WORLD_SIZE={world_env} set by the launcher")
    if args.impl == "reference":
        run_reference(args)
    elif args.shard_replicas:
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
