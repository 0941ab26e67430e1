"""Device-side fill of the seeded generator (csrc/fill.cu), for workloads too large to stage from the host.

Produces bit-for-bit the values of ``generator.fill_f32`` / ``generator.fill_bf16_bits``.
"""
from __future__ import annotations

import ctypes as C
import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "fill.cu")
LIB_PATH = os.path.join(HERE, "lib", "libhdet_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= os.path.getmtime(SRC):
        return LIB_PATH
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    os.makedirs(os.path.dirname(LIB_PATH), exist_ok=True)
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "--shared", "-Xcompiler", "-fPIC",
           "-cudart", "static", SRC, "-o", LIB_PATH]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB_PATH


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run hdet_inputs.device.build()")
        _lib = C.CDLL(LIB_PATH)
        _lib.hdet_inputs_fill.argtypes = [C.c_void_p, C.c_longlong, C.c_ulonglong, C.c_ulonglong, C.c_float,
                                          C.c_int, C.c_void_p]
        _lib.hdet_inputs_fill.restype = C.c_int
    return _lib


def fill(tensor, key: int, start: int, scale, stream: int = 0) -> None:
    """Fills a contiguous CUDA tensor (float32 or bfloat16) with generator values for indices start .. start+numel-1."""
    import torch

    if not tensor.is_cuda or not tensor.is_contiguous():
        raise ValueError("fill needs a contiguous CUDA tensor")
    dtype = {torch.float32: 0, torch.bfloat16: 1}[tensor.dtype]
    err = _load().hdet_inputs_fill(tensor.data_ptr(), tensor.numel(), key, start, float(scale), dtype, stream)
    if err != 0:
        raise RuntimeError(f"hdet_inputs_fill: CUDA error {err}")
