"""Seeded synthetic inputs shared by the CUDA library's tests, the benchmark and the CPU oracle.

Holds the integer generator (numpy here, CUDA in ``csrc/fill.cu``), the workload
recipes and nothing of the method itself.
"""
from . import generator, recipes, workloads  # noqa: F401
