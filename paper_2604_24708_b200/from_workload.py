"""Marshals a workload recipe (any object with the fields of hdet_inputs.workloads.Workload) into the C structs."""
from __future__ import annotations

from . import binding as B


def config_for(w, fuse: int = 1, device: int = 0, grad_mode: int = 0, n_local: int = 0, replica_offset: int = 0) -> B.hdet_config:
    """n_local > 0: the handle holds replicas replica_offset .. replica_offset + n_local - 1 of w.n_replicas."""
    return B.hdet_config(
        n_replicas=n_local or w.n_replicas, n_replicas_global=w.n_replicas if n_local else 0,
        replica_offset=replica_offset if n_local else 0, n_groups=w.n_groups, optimizer=w.optimizer, grad_dtype=w.grad_dtype,
        beta1=w.beta1, beta2=w.beta2, eps=w.eps, momentum=getattr(w, "momentum", 0.0), alpha_lr=w.alpha_lr, alpha_wd=w.alpha_wd,
        sync_interval=w.sync_interval, reshuffle=w.reshuffle, fuse_converge=fuse, seed=w.seed, device=device,
        grad_mode=grad_mode)


def schedule_for(w) -> B.hdet_schedule:
    return B.make_schedule(
        w.sched_kind, w.total_steps, list(w.max_lr), list(w.weight_decay), pct_start=w.pct_start,
        div_factor=w.div_factor, final_div_factor=w.final_div_factor, autolr=w.autolr,
        warmup_steps=w.warmup_steps, beta=w.ctrl_beta, sigma=w.ctrl_sigma, lambda_=w.ctrl_lambda,
        f_div=w.f_div, f_final=w.f_final, auto_wd=getattr(w, "auto_wd", 0))
