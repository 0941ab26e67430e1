"""Per-workload input recipes built on the integer generator.

Index domain: the element offset inside one replica's arena (see
``Workload.arena_offsets``).  Streams:

* initial parameters: N(0, param_sigma^2), fp32, the same for every replica;
* gradients: N(0, grad_sigma^2), regenerated per step and per replica, fp32 or
  bf16 (the bf16 value is what both sides consume, widened exactly);
* per-replica losses, host doubles: "uniform" = U(2, 3); "rank" =
  3.0 - 0.1 * offset_r + N(0, 0.01^2), where offset_r in [-1, 1] is the position
  of replica r's current learning-rate multiplier inside the spread (lowest -1,
  highest +1), so a replica that holds a higher learning rate reports a lower loss.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from . import generator as G
from .workloads import DTYPE_BF16, Workload


def param_key(w: Workload) -> int:
    return G.stream_key(w.seed, G.STREAM_PARAM, 0, 0)


def grad_key(w: Workload, step: int, replica: int) -> int:
    return G.stream_key(w.seed, G.STREAM_GRAD, step, replica)


def param_scale(w: Workload) -> np.float32:
    return G.scale_for_sigma(w.param_sigma)


def grad_scale(w: Workload) -> np.float32:
    return G.scale_for_sigma(w.grad_sigma)


def param_slab(w: Workload, start: int, n: int) -> np.ndarray:
    """Initial fp32 parameters for arena elements start .. start+n-1 (any replica)."""
    return G.fill_f32(param_key(w), start, n, param_scale(w))


def grad_slab(w: Workload, step: int, replica: int, start: int, n: int) -> np.ndarray:
    """Gradient values, as fp32 (bf16 gradients are returned widened exactly)."""
    key = grad_key(w, step, replica)
    if w.grad_dtype == DTYPE_BF16:
        return G.fill_bf16_as_f32(key, start, n, grad_scale(w))
    return G.fill_f32(key, start, n, grad_scale(w))


def rank_offsets(perm: Sequence[int]) -> np.ndarray:
    """Position of each replica's multiplier inside the spread, mapped to [-1, 1]."""
    n = len(perm)
    half = (n - 1) / 2.0
    return (np.asarray(perm, dtype=np.float64) - half) / max(half, 0.5)


def step_losses(w: Workload, step: int, perm_group0: Optional[Sequence[int]] = None) -> np.ndarray:
    """Per-replica losses (double) reported at 0-based step ``step``."""
    n = w.n_replicas
    key = G.stream_key(w.seed, G.STREAM_LOSS, step, 0)
    if w.loss_kind == "uniform":
        return 2.0 + G.uniform01(key, 0, n)
    if w.loss_kind == "rank":
        perm = list(range(n)) if perm_group0 is None else perm_group0
        return 3.0 - 0.1 * rank_offsets(perm) + 0.01 * G.standard_normal(key, 0, n)
    raise ValueError(f"unknown loss_kind {w.loss_kind!r}")
