"""Drives the CPU oracle over chosen element ranges of a synthetic workload.

THIS IS TEST INFRASTRUCTURE, like the oracle itself: it is imported by tests/, by the smoke run and by
the CPU-baseline / reference legs of bench.py, never by the CUDA library's package.  It holds none
of the method's arithmetic: it cuts a workload into slabs, feeds the oracle the seeded inputs of
those slabs (hdet_inputs), and compares arrays.  The path is independent per element, so the oracle
can run on any subset of the elements through all steps; that is what keeps the 1.3 B-parameter
workload (250 GB in double precision) within reach of a CPU.

``OracleRun``   one oracle over a list of slabs, in this process.
``OraclePool``  the same slabs split over worker processes (started with ``spawn``: a process forked
                after the first CUDA call hangs), each running its own ``OracleRun``.
"""
from __future__ import annotations

import multiprocessing as mp
import os
from types import SimpleNamespace
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from hdet_inputs import recipes as R
from hdet_inputs import workloads as W
from oracle import hdet_oracle as O

Slab = Tuple[int, int, int]   # (tensor index, first element inside the tensor, length)
TILE = 2048                   # sampling granularity (the library's tile; any value gives a valid sample)


# ----------------------------------------------------------------------------- slabs
def whole_tensor_slabs(w: W.Workload) -> List[Slab]:
    return [(k, 0, t.numel) for k, t in enumerate(w.tensors)]


def edge_slabs(w: W.Workload, tile: int = TILE) -> List[Slab]:
    """First tile and last tile (with the ragged tail) of EVERY tensor; tensors of up to two tiles whole."""
    out: List[Slab] = []
    for k, t in enumerate(w.tensors):
        n = t.numel
        if n <= 2 * tile:
            out.append((k, 0, n))
            continue
        out.append((k, 0, tile))
        last = max(tile, (n - 1) // tile * tile - tile)      # the last full tile together with the ragged tail
        out.append((k, last, n - last))
    return out


def random_run_slabs(w: W.Workload, fraction: float, run_tiles: int = 64, tile: int = TILE, seed: int = 0) -> List[Slab]:
    """Disjoint runs of `run_tiles` consecutive tiles at random positions, at least `fraction` of all elements.

    Every tensor is cut into aligned runs; a run is drawn with probability proportional to its length until the
    quota is met, so large and small tensors are both reached.
    """
    rng = np.random.default_rng(seed)
    runs: List[Slab] = []
    for k, t in enumerate(w.tensors):
        step = run_tiles * tile
        for s in range(0, t.numel, step):
            runs.append((k, s, min(step, t.numel - s)))
    order = rng.permutation(len(runs))
    need = fraction * w.numel
    out, have = [], 0
    for j in order:
        if have >= need:
            break
        out.append(runs[int(j)])
        have += runs[int(j)][2]
    return sorted(out)


def slab_elements(slabs: Sequence[Slab]) -> int:
    return int(sum(n for (_, _, n) in slabs))


# ----------------------------------------------------------------------------- one oracle
def oracle_for(w: W.Workload, params: Sequence[np.ndarray], groups: Sequence[int],
               grad_mean: bool = False) -> O.HdetOracle:
    return O.HdetOracle(
        params, groups, w.n_groups, optimizer=w.optimizer, total_steps=w.total_steps, sched_kind=w.sched_kind,
        max_lr=list(w.max_lr), weight_decay=list(w.weight_decay), pct_start=w.pct_start, div_factor=w.div_factor,
        final_div_factor=w.final_div_factor, alpha_lr=w.alpha_lr, alpha_wd=w.alpha_wd,
        sync_interval=w.sync_interval, autolr=bool(w.autolr), warmup_steps=w.warmup_steps, ctrl_beta=w.ctrl_beta,
        ctrl_sigma=w.ctrl_sigma, ctrl_lambda=w.ctrl_lambda, f_div=w.f_div, f_final=w.f_final,
        reshuffle=bool(w.reshuffle), seed=w.seed, beta1=w.beta1, beta2=w.beta2, eps=w.eps, n_replicas=w.n_replicas,
        grad_mean=grad_mean, momentum=w.momentum, auto_wd=bool(w.auto_wd))


class OracleRun:
    """The oracle over chosen element ranges (slabs) of the workload, with the same seeded inputs."""

    def __init__(self, w: W.Workload, slabs: Sequence[Slab], shared_grad: bool = False, grad_mean: bool = False,
                 loss_dtype: str = "float64"):
        self.w, self.slabs, self.shared_grad = w, list(slabs), shared_grad
        self.loss_dtype = loss_dtype
        offs = w.arena_offsets()
        self.starts = [offs[k] + s for (k, s, n) in self.slabs]
        params = [np.tile(R.param_slab(w, a, n).astype(np.float64), (w.n_replicas, 1))
                  for a, (k, s, n) in zip(self.starts, self.slabs)]
        self.o = oracle_for(w, params, [w.tensors[k].group for (k, s, n) in self.slabs], grad_mean=grad_mean)
        self.i = 0

    def grads(self, step: int) -> List[np.ndarray]:
        w = self.w
        out = []
        for a, (k, s, n) in zip(self.starts, self.slabs):
            if self.shared_grad:
                out.append(R.grad_slab(w, step, 0, a, n).astype(np.float64))
            else:
                out.append(np.stack([R.grad_slab(w, step, r, a, n) for r in range(w.n_replicas)]).astype(np.float64))
        return out

    def step(self) -> bool:
        losses = R.step_losses(self.w, self.i, self.o.perm_lr[0])
        if self.loss_dtype == "float32":           # what the library reads from an fp32 loss tensor, exactly
            losses = losses.astype(np.float32).astype(np.float64)
        ended = self.o.step(self.grads(self.i), losses)
        self.i += 1
        return ended


# ----------------------------------------------------------------------------- comparison
def rel_err(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """|got - ref| / max(|ref|, RMS(ref)): per-element relative error with an RMS floor near zero."""
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    return np.abs(np.asarray(got, dtype=np.float64) - ref) / den


SCALAR_FIELDS = ("base", "vel", "ctrl_base", "delta", "lr", "wd", "wd_base", "vel_wd", "perm_lr", "perm_wd",
                 "fired", "w", "loss_round")


def scalar_snapshot(o: O.HdetOracle) -> SimpleNamespace:
    """The oracle's schedule / spread / controller scalars as a small picklable object."""
    snap = SimpleNamespace()
    for name in SCALAR_FIELDS:
        if hasattr(o, name):
            v = getattr(o, name)
            setattr(snap, name, None if v is None else (np.array(v).tolist() if not isinstance(v, (bool, int, float)) else v))
    return snap


def _arrays_of(run: OracleRun, idx: int) -> Dict[str, np.ndarray]:
    out = {"param": run.o.theta[idx]}
    if run.w.optimizer == W.OPT_ADAMW:
        out["m"], out["v"] = run.o.m[idx], run.o.v[idx]
    elif run.w.momentum != 0.0:
        out["m"] = run.o.m[idx]
    return out


def compare_run(run: OracleRun, got: Sequence[Dict[str, np.ndarray]], tol: float) -> Tuple[float, Optional[str]]:
    """Largest relative error of `got[idx][name]` ([N, n] arrays, one dict per slab) against the oracle's slabs.

    Returns (worst, message); message is None when every error is within tol.
    """
    worst, msg = 0.0, None
    for idx, (k, s, n) in enumerate(run.slabs):
        for name, ref in _arrays_of(run, idx).items():
            e = float(rel_err(got[idx][name], ref).max())
            if e > tol and msg is None:
                msg = f"{name} of tensor {k} [{s}:{s + n}] at step {run.i}: rel err {e:.3e} > {tol:.1e}"
            worst = max(worst, e)
    return worst, msg


# ----------------------------------------------------------------------------- worker processes
def _worker_main(conn, w, slabs, kwargs):
    run = OracleRun(w, slabs, **kwargs)
    conn.send(("ready", len(slabs)))
    while True:
        cmd, arg = conn.recv()
        if cmd == "step":
            ended = False
            for _ in range(arg):
                ended = run.step()
            conn.send((ended, run.o.perm_lr[0]))
        elif cmd == "scalars":
            conn.send(scalar_snapshot(run.o))
        elif cmd == "compare":
            got, tol = arg
            conn.send(compare_run(run, got, tol))
        elif cmd == "time_steps":          # the CPU-baseline leg: `arg` steps with the gradients of step 0 held fixed
            import time
            grads = run.grads(0)
            losses = R.step_losses(run.w, 0, run.o.perm_lr[0])
            conn.recv()                    # start signal, so that all workers run at the same time
            t0 = time.perf_counter()
            for _ in range(arg):
                run.o.step(grads, losses)
            conn.send(time.perf_counter() - t0)
        elif cmd == "close":
            conn.close()
            return


def usable_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


class OraclePool:
    """The slabs split over `n_workers` spawned processes (balanced by element count), stepped in lockstep."""

    def __init__(self, w: W.Workload, slabs: Sequence[Slab], n_workers: Optional[int] = None, **kwargs):
        self.w, self.slabs = w, list(slabs)
        n_workers = max(1, min(n_workers or usable_cores(), len(self.slabs)))
        # largest slabs first, each to the least loaded worker
        load = [0] * n_workers
        self.assign: List[List[int]] = [[] for _ in range(n_workers)]
        for idx in sorted(range(len(self.slabs)), key=lambda j: -self.slabs[j][2]):
            j = load.index(min(load))
            self.assign[j].append(idx)
            load[j] += self.slabs[idx][2]
        for a in self.assign:
            a.sort()
        ctx = mp.get_context("spawn")
        self.conns, self.procs = [], []
        for a in self.assign:
            parent, child = ctx.Pipe()
            p = ctx.Process(target=_worker_main, args=(child, w, [self.slabs[j] for j in a], kwargs), daemon=True)
            p.start()
            child.close()
            self.conns.append(parent)
            self.procs.append(p)
        for c in self.conns:
            assert c.recv()[0] == "ready"
        self.i = 0
        self.n_workers = n_workers

    def _all(self, cmd, args=None):
        for j, c in enumerate(self.conns):
            c.send((cmd, args[j] if isinstance(args, list) else args))
        return [c.recv() for c in self.conns]

    def step(self, count: int = 1) -> Tuple[bool, List[int]]:
        """Advances every worker by `count` updates; returns (a round just ended, permutation of group 0)."""
        res = self._all("step", count)
        assert all(r == res[0] for r in res), "workers disagree on the scalar trajectory"
        self.i += count
        return res[0][0], list(res[0][1])

    def scalars(self) -> SimpleNamespace:
        self.conns[0].send(("scalars", None))
        return self.conns[0].recv()

    def compare(self, fetch, tol: float) -> float:
        """fetch(k, start, n) -> {"param": [N, n], "m": ..., "v": ...} for one slab; asserts every error <= tol."""
        args = [([fetch(*self.slabs[j]) for j in a], tol) for a in self.assign]
        res = self._all("compare", args)
        for worst, msg in res:
            assert msg is None, msg
        return max(r[0] for r in res)

    def time_steps(self, steps: int) -> float:
        """Wall time of `steps` oracle steps on every worker at once (gradients held fixed)."""
        import time
        for c in self.conns:
            c.send(("time_steps", steps))
        t0 = time.perf_counter()
        for c in self.conns:
            c.send("go")
        for c in self.conns:
            c.recv()
        return time.perf_counter() - t0

    def close(self):
        for c in self.conns:
            try:
                c.send(("close", None))
            except (BrokenPipeError, OSError):
                pass
        for p in self.procs:
            p.join(timeout=10)
            if p.is_alive():
                p.terminate()
        self.conns, self.procs = [], []


def one_step_errors(args) -> Tuple[float, Optional[str]]:
    """Worker function (picklable): the oracle's FIRST update on `slabs` from the seeded initial state, compared
    with the values in `got` (one dict of [N, n] arrays per slab)."""
    w, slabs, got, tol, kwargs = args
    run = OracleRun(w, slabs, **kwargs)
    run.step()
    return compare_run(run, got, tol)
