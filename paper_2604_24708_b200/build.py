"""Builds libhdet.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libhdet.so")
SOURCES = ["hdet_api.cu", "hdet_kernels.cu", "hdet_device_state.cu", "hdet_noalloc.cu", "hdet_warm.cu"]
HEADERS = ["hdet_kernels.cuh", "hdet_device_state.cuh", "hdet_scalars.h", "hdet_internal.h", os.path.join("..", "..", "include", "hdet.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-cudart", "static",
]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: libhdet.so cannot be built")
    return cand


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library if it is missing or older than its sources; returns its path."""
    if not force and not needs_build():
        return LIB_PATH
    os.makedirs(LIB_DIR, exist_ok=True)
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB_PATH]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return LIB_PATH


def ptxas_table() -> str:
    """Compiles with `-Xptxas -v` (into a scratch file, the library is left alone) and returns a markdown table:
    registers, spill bytes, stack and static shared memory of every kernel (names demangled with c++filt)."""
    import re
    import tempfile
    with tempfile.TemporaryDirectory() as tmp:
        cmd = [_nvcc()] + NVCC_FLAGS + ["-Xptxas", "-v"] + [os.path.join(CSRC, s) for s in SOURCES] + \
              ["-o", os.path.join(tmp, "scratch.so")]
        res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    rows, name = [], None
    stack = spill_st = spill_ld = 0
    for line in res.stderr.splitlines():
        m = re.search(r"Compiling entry function '([^']+)'", line)
        if m:
            name = m.group(1)
            stack = spill_st = spill_ld = 0
            continue
        m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
        if m and name:
            stack, spill_st, spill_ld = map(int, m.groups())
            continue
        m = re.search(r"Used (\d+) registers(?:, used (\d+) barriers)?(?:.*?(\d+) bytes smem)?", line)
        if m and name:
            rows.append((name, int(m.group(1)), spill_st, spill_ld, stack, int(m.group(3) or 0)))
            name = None
    try:
        dem = subprocess.run(["c++filt"], input="\n".join(r[0] for r in rows), capture_output=True, text=True).stdout.splitlines()
    except OSError:
        dem = [r[0] for r in rows]
    out = ["| kernel | registers | spill stores (B) | spill loads (B) | stack (B) | static smem (B) |", "|---|---|---|---|---|---|"]
    for (raw, regs, st, ld, stk, smem), nm in zip(rows, dem):
        nm = re.sub(r"hdet::\(anonymous namespace\)::|\(anonymous namespace\)::", "", nm)
        nm = re.sub(r"\(hdet::LaunchPlan.*$|\(.*$", "", nm).replace("void ", "")
        out.append(f"| `{nm}` | {regs} | {st} | {ld} | {stk} | {smem} |")
    return "\n".join(out)


if __name__ == "__main__":
    if "--ptxas-table" in sys.argv:
        print(ptxas_table())
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
