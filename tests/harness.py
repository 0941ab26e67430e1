"""Shared test harness: drives the CUDA library and the CPU oracle with the same seeded inputs."""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

from hdet_inputs import recipes as R
from hdet_inputs import workloads as W
from oracle import hdet_oracle as O
# The oracle's driver (slab selection, seeded inputs, worker processes, error measure) lives beside the oracle.
from oracle.driver import (OraclePool, OracleRun, Slab, edge_slabs, oracle_for, random_run_slabs,  # noqa: F401
                           rel_err, slab_elements, whole_tensor_slabs)


# ----------------------------------------------------------------------------- library side
def lib_config(B, w: W.Workload, fuse: int = 1, device: int = 0, grad_mode: int = 0):
    from paper_2604_24708_b200 import from_workload
    return from_workload.config_for(w, fuse, device, grad_mode)


def lib_schedule(B, w: W.Workload):
    from paper_2604_24708_b200 import from_workload
    return from_workload.schedule_for(w)


class GpuRun:
    """The workload resident on the GPU, stepped through the C ABI."""

    def __init__(self, w: W.Workload, fuse: int = 1, shared_grad: bool = False, device: int = 0,
                 grad_mean: bool = False, shared_state: bool = False, device_resident: bool = False,
                 loss_dtype: str = "float64", bf16_copy: bool = False):
        import torch
        from hdet_inputs import device as D
        from paper_2604_24708_b200 import binding as B
        from paper_2604_24708_b200.arena import StackedArena

        self.B, self.D, self.torch, self.w = B, D, torch, w
        self.arena = StackedArena([t.numel for t in w.tensors], [t.group for t in w.tensors], w.n_replicas,
                                  w.optimizer, w.grad_dtype, device=f"cuda:{device}", align_elems=w.align_elems,
                                  shared_grad=shared_grad, shared_state=shared_state,
                                  sgd_momentum=(w.optimizer == W.OPT_SGD and w.momentum != 0.0), bf16_copy=bf16_copy)
        assert self.arena.offsets == w.arena_offsets()
        D.fill(self.arena.param[0], R.param_key(w), 0, R.param_scale(w))
        for r in range(1, w.n_replicas):
            self.arena.param[r].copy_(self.arena.param[0])
        self.h = B.hdet_create(lib_config(B, w, fuse, device, 1 if grad_mean else 0), self.arena.descriptors())
        B.hdet_set_schedule(self.h, lib_schedule(B, w))
        self.i = 0
        self.device_resident = device_resident
        self.loss_buf = torch.zeros(w.n_replicas, dtype=getattr(torch, loss_dtype), device=f"cuda:{device}")

    def fill_grads(self, step: int) -> None:
        a, w = self.arena, self.w
        if a.shared_grad:
            self.D.fill(a.grad, R.grad_key(w, step, 0), 0, R.grad_scale(w))
        else:
            for r in range(w.n_replicas):
                self.D.fill(a.grad[r], R.grad_key(w, step, r), 0, R.grad_scale(w))

    def perm0(self) -> List[int]:
        st = self.B.hdet_get_state(self.h)
        return list(st.perm_lr[0])[: self.w.n_replicas]

    def step(self, perm0: Optional[Sequence[int]] = None) -> bool:
        """One update with regenerated gradients and recipe losses; runs the controller after a sync."""
        self.fill_grads(self.i)
        losses = R.step_losses(self.w, self.i, perm0)
        if self.device_resident:
            # the losses stay on the device; the controller runs there too
            self.loss_buf.copy_(self.torch.from_numpy(np.asarray(losses)).to(self.loss_buf.dtype))
            ended = self.B.hdet_step_device(self.h, self.loss_buf, self.torch.cuda.current_stream().cuda_stream)
        else:
            ended = self.B.hdet_step(self.h, list(losses))
            if ended:
                self.B.hdet_autolr_update(self.h)
        self.i += 1
        return ended

    def state(self):
        return self.B.hdet_get_state(self.h)

    def slab(self, which: str, k: int, start: int, n: int) -> np.ndarray:
        """[N, n] values of tensor k, elements start .. start+n-1, copied to the host."""
        t = {"param": self.arena.param, "m": self.arena.exp_avg, "v": self.arena.exp_avg_sq}[which]
        off = self.arena.offsets[k] + start
        if t.dim() == 1:                       # moments shared by all replicas
            return t[None, off:off + n].float().cpu().numpy()
        return t[:, off:off + n].float().cpu().numpy()

    def close(self) -> None:
        self.torch.cuda.synchronize()
        self.B.hdet_destroy(self.h)
        self.h = None
        self.arena = None
        self.torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- comparison
def compare_slabs(g: GpuRun, o: OracleRun, tol: float, check_moments: bool = True) -> float:
    """Largest relative error over all slabs (params and, for AdamW, both moments); asserts it is <= tol."""
    worst = 0.0
    adam = g.w.optimizer == W.OPT_ADAMW
    for idx, (k, s, n) in enumerate(o.slabs):
        pairs = [("param", o.o.theta[idx])]
        if adam and check_moments:
            pairs += [("m", o.o.m[idx]), ("v", o.o.v[idx])]
        if g.w.optimizer == W.OPT_SGD and g.w.momentum != 0.0 and check_moments:
            pairs += [("m", o.o.m[idx])]
        for name, ref in pairs:
            got = g.slab(name, k, s, n)
            if got.shape[0] == 1 and ref.shape[0] > 1:       # shared moments: every oracle replica must agree
                assert np.all(ref == ref[0:1]), f"oracle {name} differs between replicas although the gradient is common"
                ref = ref[0:1]
            e = rel_err(got, ref).max()
            assert e <= tol, f"{name} of tensor {k} [{s}:{s + n}] at step {g.i}: rel err {e:.3e} > {tol:.1e}"
            worst = max(worst, float(e))
    return worst


def compare_scalars(st, o: O.HdetOracle, n: int, G: int, tol: float = 1e-12) -> None:
    """Schedule / spread / controller scalars of the library against the oracle (relative 1e-12)."""
    def close(a, b, what):
        a, b = float(a), float(b)
        assert abs(a - b) <= tol * max(abs(b), 1e-300) or abs(a - b) < 1e-300, f"{what}: {a!r} vs {b!r}"
    for g in range(G):
        close(st.base[g], o.base[g], f"base[{g}]")
        assert abs(float(st.velocity[g]) - o.vel[g]) <= tol * max(abs(o.base[g]), 1e-300), f"velocity[{g}]"
        if o.fired:
            close(st.ctrl_base[g], o.ctrl_base[g], f"ctrl_base[{g}]")
            a, b = float(st.delta[g]), float(o.delta[g])
            assert abs(a - b) <= tol * max(abs(o.base[g]), 1e-300), f"delta[{g}]: {a!r} vs {b!r}"
        for r in range(n):
            close(st.lr[g][r], o.lr[g][r], f"lr[{g}][{r}]")
            close(st.wd[g][r], o.wd[g][r], f"wd[{g}][{r}]")
        close(st.wd_base[g], o.wd_base[g], f"wd_base[{g}]")
        assert abs(float(st.wd_velocity[g]) - o.vel_wd[g]) <= tol * max(abs(o.wd_base[g]), 1e-300), f"wd_velocity[{g}]"
        assert list(st.perm_lr[g])[:n] == o.perm_lr[g], f"perm_lr[{g}]"
        assert list(st.perm_wd[g])[:n] == o.perm_wd[g], f"perm_wd[{g}]"
    assert bool(st.fired) == o.fired
    if o.w is not None:
        for r in range(n):
            close(st.weights[r], o.w[r], f"w[{r}]")
