"""ctypes binding of libhdet (include/hdet.h): same names, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; nothing here computes.
There is no fallback: if the shared library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

HDET_MAX_REPLICAS = 32
HDET_MAX_GROUPS = 8

HDET_OK = 0
HDET_ERR_INVALID_ARG = 1
HDET_ERR_STATE = 2
HDET_ERR_ALIGN = 3
HDET_ERR_UNSUPPORTED = 4
HDET_ERR_CUDA = 5
HDET_ERR_NONFINITE = 6
HDET_ERR_TIMEOUT = 7

HDET_OPT_SGD, HDET_OPT_ADAMW = 0, 1
HDET_DTYPE_F32, HDET_DTYPE_BF16, HDET_DTYPE_F64 = 0, 1, 2
HDET_GRAD_AS_GIVEN, HDET_GRAD_REPLICA_MEAN = 0, 1
HDET_SCHED_CONSTANT, HDET_SCHED_ONECYCLE_COS, HDET_SCHED_ONECYCLE_LINEAR = 0, 1, 2

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libhdet.so")


class HdetError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"hdet status {status}: {message}")
        self.status = status
        self.message = message


class hdet_tensor(C.Structure):
    _fields_ = [
        ("param", C.c_void_p), ("grad", C.c_void_p), ("exp_avg", C.c_void_p), ("exp_avg_sq", C.c_void_p),
        ("numel", C.c_int64), ("param_stride", C.c_int64), ("grad_stride", C.c_int64), ("state_stride", C.c_int64),
        ("group", C.c_int32), ("reserved", C.c_int32), ("param_bf16", C.c_void_p),
    ]


class hdet_config(C.Structure):
    _fields_ = [
        ("n_replicas", C.c_int32), ("n_groups", C.c_int32), ("optimizer", C.c_int32), ("grad_dtype", C.c_int32),
        ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double), ("momentum", C.c_double),
        ("alpha_lr", C.c_double), ("alpha_wd", C.c_double), ("sync_interval", C.c_int64),
        ("reshuffle", C.c_int32), ("fuse_converge", C.c_int32), ("seed", C.c_uint64),
        ("device", C.c_int32), ("grad_mode", C.c_int32),
        ("n_replicas_global", C.c_int32), ("replica_offset", C.c_int32),
    ]


class hdet_schedule(C.Structure):
    _fields_ = [
        ("kind", C.c_int32), ("autolr", C.c_int32), ("total_steps", C.c_int64),
        ("max_lr", C.POINTER(C.c_double)), ("weight_decay", C.POINTER(C.c_double)),
        ("pct_start", C.c_double), ("div_factor", C.c_double), ("final_div_factor", C.c_double),
        ("warmup_steps", C.c_int64), ("beta", C.c_double), ("sigma", C.c_double), ("lambda_", C.c_double),
        ("f_div", C.c_double), ("f_final", C.c_double), ("auto_wd", C.c_int32), ("reserved", C.c_int32),
    ]


_GD = C.c_double * HDET_MAX_GROUPS
_ND = C.c_double * HDET_MAX_REPLICAS
_GND = (C.c_double * HDET_MAX_REPLICAS) * HDET_MAX_GROUPS
_GNI = (C.c_int32 * HDET_MAX_REPLICAS) * HDET_MAX_GROUPS


class hdet_state(C.Structure):
    _fields_ = [
        ("step", C.c_int64), ("n_acc", C.c_int64), ("fired", C.c_int32), ("round_ended", C.c_int32),
        ("device_status", C.c_uint32), ("reserved", C.c_int32),
        ("base", _GD), ("ctrl_base", _GD), ("velocity", _GD), ("delta", _GD),
        ("lr", _GND), ("wd", _GND), ("perm_lr", _GNI), ("perm_wd", _GNI),
        ("weights", _ND), ("loss_acc", _ND), ("loss_round", _ND), ("gamma", C.c_double),
        ("wd_base", _GD), ("wd_velocity", _GD), ("wd_delta", _GD),
    ]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2604_24708_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    H = C.c_void_p
    lib.hdet_create.argtypes = [C.POINTER(hdet_config), C.POINTER(hdet_tensor), C.c_int64, C.POINTER(H)]
    lib.hdet_set_schedule.argtypes = [H, C.POINTER(hdet_schedule)]
    lib.hdet_step.argtypes = [H, C.POINTER(C.c_double), C.c_void_p, C.POINTER(C.c_int32)]
    lib.hdet_step_device.argtypes = [H, C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(C.c_int32)]
    lib.hdet_step_device.restype = C.c_int
    lib.hdet_step_host_grads.argtypes = [H, C.POINTER(C.c_void_p), C.POINTER(C.c_double), C.c_void_p,
                                         C.POINTER(C.c_int32)]
    lib.hdet_step_host_grads.restype = C.c_int
    lib.hdet_step_sharded.argtypes = [H, C.POINTER(C.c_double), C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.hdet_step_sharded.restype = C.c_int
    lib.hdet_apply_mean.argtypes = [H, C.c_void_p, C.c_void_p]
    lib.hdet_apply_mean.restype = C.c_int
    lib.hdet_apply_mean_peers.argtypes = [H, C.POINTER(C.c_void_p), C.c_int32, C.c_void_p]
    lib.hdet_apply_mean_peers.restype = C.c_int
    lib.hdet_partial_layout.argtypes = [H, C.POINTER(C.c_int64), C.c_int64, C.POINTER(C.c_int64)]
    lib.hdet_partial_layout.restype = C.c_int
    lib.hdet_warm_init.argtypes = [H, C.c_double, C.c_uint64, C.c_void_p]
    lib.hdet_warm_init.restype = C.c_int
    lib.hdet_converge.argtypes = [H, C.c_void_p]
    lib.hdet_autolr_update.argtypes = [H, C.POINTER(C.c_double), C.c_void_p]
    lib.hdet_get_state.argtypes = [H, C.POINTER(hdet_state)]
    lib.hdet_set_state.argtypes = [H, C.POINTER(hdet_state)]
    lib.hdet_destroy.argtypes = [H]
    lib.hdet_last_error.argtypes = [H]
    lib.hdet_last_error.restype = C.c_char_p
    lib.hdet_kernel_launches.argtypes = [H]
    lib.hdet_kernel_launches.restype = C.c_int64
    lib.hdet_converge_static.argtypes = [C.POINTER(hdet_tensor), C.c_int64, C.c_int32, C.c_int32, C.c_void_p]
    lib.hdet_converge_static.restype = C.c_int
    lib.hdet_plan_tiles.argtypes = [C.POINTER(hdet_config), C.POINTER(hdet_tensor), C.c_int64, C.POINTER(C.c_int32),
                                    C.POINTER(C.c_int32), C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int32),
                                    C.POINTER(C.c_int64)]
    lib.hdet_plan_tiles.restype = C.c_int
    lib.hdet_selftest_bounded_wait.argtypes = [H, C.c_void_p]
    lib.hdet_selftest_bounded_wait.restype = C.c_int
    for f in ("hdet_create", "hdet_set_schedule", "hdet_step", "hdet_converge", "hdet_autolr_update",
              "hdet_get_state", "hdet_set_state", "hdet_destroy"):
        getattr(lib, f).restype = C.c_int
    return lib


_lib = _load()


def _check(status: int, handle) -> None:
    if status != HDET_OK:
        msg = _lib.hdet_last_error(handle)
        raise HdetError(status, msg.decode() if msg else "")


def _doubles(values: Optional[Sequence[float]]):
    if values is None:
        return None
    return (C.c_double * len(values))(*[float(v) for v in values])


def tensor_from_torch(param, grad, exp_avg=None, exp_avg_sq=None, group: int = 0) -> hdet_tensor:
    """Descriptor for tensors whose first axis is the replica axis ([N, ...], inner axes contiguous).

    ``grad`` may lack the replica axis (same shape as one replica): it is then shared (stride 0).
    """
    n = param.shape[0]
    numel = param[0].numel()
    if not param[0].is_contiguous():
        raise ValueError("each replica of param must be contiguous")
    shared = grad.dim() == param.dim() - 1 or (grad.shape[0] == 1 and n > 1)
    g0 = grad if grad.dim() == param.dim() - 1 else grad[0]
    if g0.numel() != numel or not g0.is_contiguous():
        raise ValueError("grad must match one replica of param and be contiguous")
    t = hdet_tensor()
    t.param = param.data_ptr()
    t.grad = grad.data_ptr()
    t.numel = numel
    t.param_stride = param.stride(0) if n > 1 else numel
    t.grad_stride = 0 if shared else (grad.stride(0) if n > 1 else numel)
    if exp_avg is not None:
        if not (exp_avg[0].is_contiguous() and exp_avg_sq[0].is_contiguous()) or exp_avg.stride(0) != exp_avg_sq.stride(0):
            raise ValueError("moments must be contiguous per replica and share one replica stride")
        t.exp_avg = exp_avg.data_ptr()
        t.exp_avg_sq = exp_avg_sq.data_ptr()
        t.state_stride = exp_avg.stride(0) if n > 1 else numel
    t.group = group
    return t


def make_schedule(kind: int, total_steps: int, max_lr: Sequence[float], weight_decay: Optional[Sequence[float]] = None,
                  pct_start: float = 0.3, div_factor: float = 25.0, final_div_factor: float = 1e4, autolr: int = 0,
                  warmup_steps: int = 0, beta: float = 0.9, sigma: float = 0.1, lambda_: float = 0.5,
                  f_div: float = 25.0, f_final: float = 1.0, auto_wd: int = 0) -> hdet_schedule:
    s = hdet_schedule()
    s.kind, s.autolr, s.total_steps = kind, int(autolr), total_steps
    s._max_lr = _doubles(max_lr)            # keep the host arrays alive with the struct
    s._weight_decay = _doubles(weight_decay)
    s.max_lr = C.cast(s._max_lr, C.POINTER(C.c_double))
    s.weight_decay = C.cast(s._weight_decay, C.POINTER(C.c_double)) if weight_decay is not None else None
    s.pct_start, s.div_factor, s.final_div_factor = pct_start, div_factor, final_div_factor
    s.warmup_steps, s.beta, s.sigma, s.lambda_ = warmup_steps, beta, sigma, lambda_
    s.f_div, s.f_final = f_div, f_final
    s.auto_wd = int(auto_wd)
    return s


def hdet_create(cfg: hdet_config, tensors: Sequence[hdet_tensor]) -> C.c_void_p:
    arr = (hdet_tensor * len(tensors))(*tensors) if tensors else None
    h = C.c_void_p()
    status = _lib.hdet_create(C.byref(cfg), arr, len(tensors), C.byref(h))
    _check(status, None)
    return h


def hdet_set_schedule(h, sched: hdet_schedule) -> None:
    _check(_lib.hdet_set_schedule(h, C.byref(sched)), h)


def hdet_step(h, step_losses: Optional[Sequence[float]] = None, stream: int = 0) -> bool:
    """Runs one update; returns True when it ended a round (the replicas were averaged)."""
    flag = C.c_int32(0)
    _check(_lib.hdet_step(h, _doubles(step_losses), C.c_void_p(stream), C.byref(flag)), h)
    return bool(flag.value)


def hdet_step_device(h, d_step_losses=None, stream: int = 0) -> bool:
    """One device-resident update; ``d_step_losses`` is a CUDA tensor of N float32 or float64 losses (or None)."""
    flag = C.c_int32(0)
    ptr, dtype = None, HDET_DTYPE_F32
    if d_step_losses is not None:
        import torch
        if not d_step_losses.is_cuda or not d_step_losses.is_contiguous():
            raise ValueError("d_step_losses must be a contiguous CUDA tensor")
        dtype = {torch.float32: HDET_DTYPE_F32, torch.float64: HDET_DTYPE_F64}[d_step_losses.dtype]
        ptr = C.c_void_p(d_step_losses.data_ptr())
    _check(_lib.hdet_step_device(h, ptr, dtype, C.c_void_p(stream), C.byref(flag)), h)
    return bool(flag.value)


def hdet_step_host_grads(h, host_grad_ptrs: Sequence[int], step_losses: Optional[Sequence[float]] = None,
                         stream: int = 0) -> bool:
    """hdet_step with the gradients taken from host memory (one pointer per tensor, laid out like the device gradient)."""
    flag = C.c_int32(0)
    arr = (C.c_void_p * max(1, len(host_grad_ptrs)))(*host_grad_ptrs) if host_grad_ptrs else None
    _check(_lib.hdet_step_host_grads(h, arr, _doubles(step_losses), C.c_void_p(stream), C.byref(flag)), h)
    return bool(flag.value)


def hdet_step_sharded(h, step_losses, d_partial, stream: int = 0) -> bool:
    """One update of a handle that holds a shard of the replica axis; ``d_partial`` is a CUDA float32 tensor."""
    flag = C.c_int32(0)
    ptr = C.c_void_p(d_partial.data_ptr()) if d_partial is not None else None
    _check(_lib.hdet_step_sharded(h, _doubles(step_losses), ptr, C.c_void_p(stream), C.byref(flag)), h)
    return bool(flag.value)


def hdet_apply_mean(h, d_sum, stream: int = 0) -> None:
    _check(_lib.hdet_apply_mean(h, C.c_void_p(d_sum.data_ptr()), C.c_void_p(stream)), h)


def hdet_apply_mean_peers(h, d_partials, stream: int = 0) -> None:
    """Every local replica <- (sum over the ranks' staging buffers, in the given rank order) / N, read by the kernel itself."""
    ptrs = [p.data_ptr() if hasattr(p, "data_ptr") else int(p) for p in d_partials]
    arr = (C.c_void_p * len(ptrs))(*ptrs)
    _check(_lib.hdet_apply_mean_peers(h, arr, len(ptrs), C.c_void_p(stream)), h)


def hdet_partial_layout(h, n_tensors: int):
    """(offsets per tensor, total elements) of the partial-sum staging buffer."""
    offs = (C.c_int64 * max(1, n_tensors))()
    total = C.c_int64(0)
    _check(_lib.hdet_partial_layout(h, offs if n_tensors else None, n_tensors, C.byref(total)), h)
    return list(offs)[:n_tensors], int(total.value)


def hdet_plan_tiles(cfg: hdet_config, tensors: Sequence[hdet_tensor]):
    """The work plan hdet_create would build, computed on the host: (tile_tensor, tile_index, access per tensor,
    partial-sum offset per tensor)."""
    arr = (hdet_tensor * len(tensors))(*tensors) if tensors else None
    count = C.c_int64(0)
    _check(_lib.hdet_plan_tiles(C.byref(cfg), arr, len(tensors), None, None, 0, C.byref(count), None, None), None)
    n = int(count.value)
    tt, ti = (C.c_int32 * max(1, n))(), (C.c_int32 * max(1, n))()
    acc, offs = (C.c_int32 * max(1, len(tensors)))(), (C.c_int64 * max(1, len(tensors)))()
    _check(_lib.hdet_plan_tiles(C.byref(cfg), arr, len(tensors), tt, ti, n, C.byref(count), acc, offs), None)
    return list(tt)[:n], list(ti)[:n], list(acc)[:len(tensors)], list(offs)[:len(tensors)]


def hdet_selftest_bounded_wait(h, stream: int = 0) -> None:
    """Launches a kernel whose bounded wait runs out (about a second): sets the timeout bit of the status word."""
    _check(_lib.hdet_selftest_bounded_wait(h, C.c_void_p(stream)), h)


def hdet_warm_init(h, nu: float = 0.01, seed: int = 0, stream: int = 0) -> None:
    """Eq. 10: every replica <- replica 0 (the checkpoint) + Gaussian noise of relative scale nu."""
    _check(_lib.hdet_warm_init(h, nu, seed, C.c_void_p(stream)), h)


def hdet_converge(h, stream: int = 0) -> None:
    _check(_lib.hdet_converge(h, C.c_void_p(stream)), h)


HDET_STATIC_MAX_TENSORS = 1024
HDET_STATIC_MAX_TILES = 65536


def hdet_converge_static(tensors: Sequence[hdet_tensor], n_replicas: int, device: int = 0, stream: int = 0) -> None:
    """Replica mean of every listed tensor without a handle and without any device allocation.

    For callers that cannot allocate at that point (all device memory owned by a framework pool, or a
    loop that must not risk the synchronisation an allocation can cause).  The work tables go into a
    static device array shared by all calls, so calls that overlap on the GPU must be serialised.
    """
    arr = (hdet_tensor * len(tensors))(*tensors) if tensors else None
    _check(_lib.hdet_converge_static(arr, len(tensors), n_replicas, device, C.c_void_p(stream)), None)


def hdet_autolr_update(h, round_losses: Optional[Sequence[float]] = None, stream: int = 0) -> None:
    _check(_lib.hdet_autolr_update(h, _doubles(round_losses), C.c_void_p(stream)), h)


def hdet_get_state(h, raise_on_nonfinite: bool = True) -> hdet_state:
    st = hdet_state()
    status = _lib.hdet_get_state(h, C.byref(st))
    if status in (HDET_ERR_NONFINITE, HDET_ERR_TIMEOUT) and not raise_on_nonfinite:   # sticky device flags: *out is filled
        return st
    _check(status, h)
    return st


def hdet_set_state(h, st: hdet_state) -> None:
    _check(_lib.hdet_set_state(h, C.byref(st)), h)


def hdet_destroy(h) -> None:
    _check(_lib.hdet_destroy(h), None)


def hdet_last_error(h=None) -> str:
    msg = _lib.hdet_last_error(h)
    return msg.decode() if msg else ""


def hdet_kernel_launches(h) -> int:
    return int(_lib.hdet_kernel_launches(h))


def raw_library() -> C.CDLL:
    """The loaded CDLL (for tests that call the C ABI with hand-built arguments)."""
    return _lib
