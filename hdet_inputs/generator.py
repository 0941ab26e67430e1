"""Seeded synthetic-input generator (CPU side, numpy).

This module produces the gradients, initial parameters and loss noise that the
tests and the benchmark feed to BOTH the CUDA library and the CPU oracle.  It
contains none of the method's arithmetic: no spread, schedule, optimizer or
controller formula lives here.

Every value is a pure function of (key, index), built from integer arithmetic
only, so the CUDA fill kernel in ``csrc/fill.cu`` reproduces it bit for bit:

    u     = mix64(key + index * GOLDEN)                 (64-bit wrap-around)
    z     = lane0(u) + lane1(u) + lane2(u) + lane3(u) - 131070
            where lane_k is the k-th 16-bit field of u  (Irwin-Hall, n = 4)
    value = fp32(z) * fp32(scale)                       (one IEEE multiply)

``z`` is an integer in [-131070, 131070] with mean 0 and standard deviation
65536/sqrt(3) * sqrt(1 - 2**-32) ~= 37837.2; fp32(z) is exact.  A bf16 value is
the fp32 value rounded to nearest-even on its bit pattern.  ``mix64`` is the
finaliser of the SplitMix64 generator (Steele, Lea & Flood, OOPSLA 2014).
"""
from __future__ import annotations

import math

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK16 = np.uint64(0xFFFF)
_U64 = (1 << 64) - 1

#: standard deviation of the integer z defined above
IRWIN_HALL_STD = math.sqrt(4.0 * (65536.0**2 - 1.0) / 12.0)

# stream identifiers (which quantity a key is for)
STREAM_PARAM = 1
STREAM_GRAD = 2
STREAM_LOSS = 3
STREAM_NOISE = 4


def mix64(x):
    """SplitMix64 finaliser on a numpy uint64 array (or scalar)."""
    x = np.asarray(x, dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * _M1
        x = (x ^ (x >> np.uint64(27))) * _M2
        x = x ^ (x >> np.uint64(31))
    return x


def _mix64_int(x: int) -> int:
    x &= _U64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _U64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _U64
    return x ^ (x >> 31)


def stream_key(seed: int, stream: int, step: int = 0, replica: int = 0) -> int:
    """64-bit key for one (seed, stream, step, replica) cell, as a Python int."""
    k = _mix64_int(seed)
    k = _mix64_int(k + stream)
    k = _mix64_int(k + step)
    k = _mix64_int(k + replica)
    return k


def scale_for_sigma(sigma: float) -> np.float32:
    """fp32 multiplier that gives the generated values standard deviation sigma."""
    return np.float32(sigma / IRWIN_HALL_STD)


def normal_int(key: int, start: int, n: int) -> np.ndarray:
    """The integers z for indices start .. start+n-1 (int32 array)."""
    idx = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        u = mix64(np.uint64(key) + idx * GOLDEN)
    s = (
        (u & _MASK16)
        + ((u >> np.uint64(16)) & _MASK16)
        + ((u >> np.uint64(32)) & _MASK16)
        + (u >> np.uint64(48))
    )
    return s.astype(np.int64).astype(np.int32) - np.int32(131070)


def fill_f32(key: int, start: int, n: int, scale: np.float32) -> np.ndarray:
    """fp32 values for indices start .. start+n-1."""
    z = normal_int(key, start, n).astype(np.float32)
    return z * np.float32(scale)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest-even on the bit pattern); returns uint16 bits.

    The generator never produces NaN or infinity, so no special cases arise.
    """
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def fill_bf16_bits(key: int, start: int, n: int, scale: np.float32) -> np.ndarray:
    """bf16 bit patterns (uint16) for indices start .. start+n-1."""
    return f32_to_bf16_bits(fill_f32(key, start, n, scale))


def fill_bf16_as_f32(key: int, start: int, n: int, scale: np.float32) -> np.ndarray:
    """The bf16 values of ``fill_bf16_bits`` widened exactly to fp32."""
    return bf16_bits_to_f32(fill_bf16_bits(key, start, n, scale))


def uniform01(key: int, start: int, n: int) -> np.ndarray:
    """Doubles in [0, 1) from the top 53 bits of mix64(key + index*GOLDEN)."""
    idx = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        u = mix64(np.uint64(key) + idx * GOLDEN)
    return (u >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def standard_normal(key: int, start: int, n: int) -> np.ndarray:
    """Approximately N(0,1) doubles: z / IRWIN_HALL_STD."""
    return normal_int(key, start, n).astype(np.float64) / IRWIN_HALL_STD
