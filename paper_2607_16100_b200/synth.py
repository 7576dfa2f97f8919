"""Seeded synthetic inputs for the AllReduce tests and the benchmark.

This module holds NO arithmetic of the AllReduce itself: it only manufactures
rank inputs.  It is the one module that the tests of the CPU oracle, the GPU
parity tests and ``bench.py`` all share, so that both sides see the same bits.

The generator is counter based: element ``i`` of rank ``q`` in call ``call`` is
a pure function of ``(seed, call, q, i)`` (a splitmix64 finaliser over a mixed
counter), so any slice of any workload can be regenerated on its own -- the
256 MiB-per-rank case is checked on sampled positions without ever holding a
second full copy.

The value distributions are those of the five benchmark workloads, which stand
in for tensor-parallel decode activations (hidden size 8192 per token, two
AllReduces per layer):

* ``int_pm8``  -- integers uniform in [-8, 8] stored as floats (sums are exact);
* ``normal``   -- N(0, 1) by Box-Muller in binary64, then rounded to the dtype;
* ``uniform``  -- U(-1, 1) from 53 random bits in binary64, then rounded.

bf16 travels as ``numpy.uint16`` bit patterns (round-to-nearest-even from fp32).
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)


def seed_for_config(k: int) -> int:
    """Base seed of benchmark workload ``k`` (1-based)."""
    return 0x5EED0000 + k


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on a uint64 array (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = z + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def raw_u64(seed: int, call: int, rank: int, idx: np.ndarray, lane: int = 0) -> np.ndarray:
    """64 random bits per index; ``lane`` selects an independent second draw."""
    with np.errstate(over="ignore"):
        key = np.uint64((seed ^ (call << 48) ^ (rank << 40) ^ (lane << 36)) & 0xFFFFFFFFFFFFFFFF)
        key = _splitmix64(np.asarray([key], dtype=np.uint64))[0]
        return _splitmix64(idx.astype(np.uint64) ^ key)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even cut of finite fp32 values to bf16 bit patterns."""
    w = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (w >> np.uint32(16)) & np.uint32(1)
    return ((w + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32)


def values_f64(dist: str, seed: int, call: int, rank: int, idx: np.ndarray) -> np.ndarray:
    """The binary64 draw at the given element indices, before rounding."""
    if dist == "int_pm8":
        u = raw_u64(seed, call, rank, idx)
        return (u % np.uint64(17)).astype(np.float64) - 8.0
    if dist == "uniform":
        u = raw_u64(seed, call, rank, idx) >> np.uint64(11)          # 53 bits
        return u.astype(np.float64) * 2.0 ** -52 - 1.0
    if dist == "normal":
        u1 = (raw_u64(seed, call, rank, idx, 0) >> np.uint64(11)).astype(np.float64)
        u2 = (raw_u64(seed, call, rank, idx, 1) >> np.uint64(11)).astype(np.float64)
        u1 = (u1 + 1.0) * 2.0 ** -53                                  # (0, 1]
        u2 = u2 * 2.0 ** -53                                          # [0, 1)
        return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    raise ValueError(f"unknown distribution {dist!r}")


def rank_slice(dist: str, dtype: str, seed: int, call: int, rank: int,
               idx: np.ndarray) -> np.ndarray:
    """Rank ``rank``'s input at element indices ``idx`` in the wire dtype
    (``float32`` for "f32", ``uint16`` bit patterns for "bf16")."""
    v = values_f64(dist, seed, call, rank, idx).astype(np.float32)
    if dtype == "f32":
        return v
    if dtype == "bf16":
        return f32_to_bf16_bits(v)
    raise ValueError(f"unknown dtype {dtype!r}")


def make_inputs(dist: str, dtype: str, P: int, count: int, seed: int, call: int = 0,
                block: int = 1 << 22, workers: int = 0) -> np.ndarray:
    """All P rank inputs as a [P, count] array, generated block by block."""
    out = np.empty((P, count), dtype=np.float32 if dtype == "f32" else np.uint16)
    jobs = [(q, lo, min(lo + block, count)) for q in range(P) for lo in range(0, count, block)]

    def fill(job):
        q, lo, hi = job
        out[q, lo:hi] = rank_slice(dist, dtype, seed, call, q,
                                   np.arange(lo, hi, dtype=np.uint64))

    if workers == 1 or len(jobs) == 1:
        for j in jobs:
            fill(j)
    else:
        import os
        with ThreadPoolExecutor(max_workers=workers or min(32, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, jobs))
    return out


# The five benchmark workloads (P, dtype, elements per rank, distribution).
WORKLOADS = {
    "c1": dict(P=4, dtype="f32", count=1024, dist="int_pm8", seed=seed_for_config(1)),
    "c2": dict(P=8, dtype="bf16", count=8192, dist="normal", seed=seed_for_config(2)),
    "c3": dict(P=8, dtype="bf16", count=8192, dist="normal", seed=seed_for_config(3),
               batch=(1, 2, 4, 8, 16, 32, 64)),
    "c4": dict(P=8, dtype="f32", count=64 << 20, dist="uniform", seed=seed_for_config(4)),
    "c5": dict(P=8, dtype="bf16", count=8192 * 4, dist="normal", seed=seed_for_config(5),
               calls=160),
}
