"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s cpu_baseline /
reference arm may import this module.  It never imports the CUDA package and
the CUDA package never imports it.

* ``allreduce``        -- the C oracle (``allreduce_oracle.c``): per element the
  binary32 sum in rank order 0..P-1, one final narrowing to the element type,
  the same value written to all P outputs (paper Sec. III-A one-shot definition,
  Sec. V ``recvReduce`` accumulator type, Table I determinism).
* ``sum_f64``          -- a second, independent reference: the sum accumulated
  in binary64 with numpy.  Not used for parity, only for the error-bound pin.
* ``gamma`` / ``error_bound`` -- the forward-error bound of Sec. IV
  ("Algorithm Comparison"): |fl(sum x) - sum x| <= gamma_{N-1} * sum |x|,
  gamma_k = k u / (1 - k u).

bf16 arrays travel as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "allreduce_oracle.c"
_LIB = _HERE / "liballreduce_oracle.so"

CFLAGS = [
    "-O2", "-fno-fast-math", "-ffp-contract=off", "-fexcess-precision=standard",
    "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall", "-Wextra",
]


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (a few hundred milliseconds)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(["gcc", *CFLAGS, "-o", str(tmp), str(_SRC)], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        for name in ("oracle_allreduce_f32", "oracle_allreduce_bf16"):
            fn = getattr(lib, name)
            fn.argtypes = [vp, vp, ci, sz]
            fn.restype = ci
        for name in ("oracle_allreduce_f32_mt", "oracle_allreduce_bf16_mt"):
            fn = getattr(lib, name)
            fn.argtypes = [vp, vp, ci, sz, ctypes.POINTER(ci)]
            fn.restype = ci
        for name in ("oracle_reduce_scatter", "oracle_all_gather", "oracle_reduce"):
            fn = getattr(lib, name)
            fn.argtypes = [vp, vp, ci, sz, ci]
            fn.restype = ci
        lib.oracle_broadcast.argtypes = [vp, vp, ci, sz, ci, ci]
        lib.oracle_broadcast.restype = ci
        lib.oracle_set_threads.argtypes = [ci]
        lib.oracle_set_threads.restype = None
        lib.oracle_narrow_bf16.argtypes = [ctypes.c_float]
        lib.oracle_narrow_bf16.restype = ctypes.c_uint16
        lib.oracle_widen_bf16.argtypes = [ctypes.c_uint16]
        lib.oracle_widen_bf16.restype = ctypes.c_float
        _lib = lib
    return _lib


def _check(x: np.ndarray) -> str:
    if x.ndim != 2:
        raise ValueError("inputs must be a [P, count] array (row q = rank q)")
    if x.dtype == np.float32:
        return "f32"
    if x.dtype == np.uint16:
        return "bf16"
    raise TypeError("dtype must be float32 or uint16 (bf16 bit patterns)")


def allreduce(x: np.ndarray, threads: int = 1) -> np.ndarray:
    """x[P, count] -> out[P, count]; row r is rank r's output.

    ``threads`` > 1 (or 0 = all host cores) splits the element loop with OpenMP;
    per-element arithmetic is identical.
    """
    out, _ = allreduce_timed_team(x, threads)
    return out


def allreduce_timed_team(x: np.ndarray, threads: int = 1):
    """As ``allreduce``; also returns the number of host threads that ran."""
    kind = _check(x)
    x = np.ascontiguousarray(x)
    P, count = x.shape
    out = np.empty_like(x)
    lib = _load()
    if threads == 1:
        fn = lib.oracle_allreduce_f32 if kind == "f32" else lib.oracle_allreduce_bf16
        rc = fn(x.ctypes.data, out.ctypes.data, P, count)
        team = 1
    else:
        _set_omp_threads(threads if threads > 0 else (os.cpu_count() or 1))
        fn = lib.oracle_allreduce_f32_mt if kind == "f32" else lib.oracle_allreduce_bf16_mt
        used = ctypes.c_int(0)
        rc = fn(x.ctypes.data, out.ctypes.data, P, count, ctypes.byref(used))
        team = used.value
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, team


# ---------------------------------------------------------------------------
# sibling collectives (Sec. V: Broadcast, Reduce, ReduceScatter, AllGather)
# ---------------------------------------------------------------------------

def reduce_scatter(x: np.ndarray) -> np.ndarray:
    """x[P, P*n] -> out[P, n]; out[r] = rank-ordered sum over q of x[q, r*n:(r+1)*n]."""
    _check(x)
    x = np.ascontiguousarray(x)
    P, total = x.shape
    if total % P:
        raise ValueError("row length must be a multiple of P")
    n = total // P
    out = np.empty((P, n), dtype=x.dtype)
    if _load().oracle_reduce_scatter(x.ctypes.data, out.ctypes.data, P, n, x.dtype.itemsize) != 0:
        raise RuntimeError("oracle_reduce_scatter failed")
    return out


def all_gather(x: np.ndarray) -> np.ndarray:
    """x[P, n] -> out[P, P*n]; every rank holds the concatenation of all inputs."""
    _check(x)
    x = np.ascontiguousarray(x)
    P, n = x.shape
    out = np.empty((P, P * n), dtype=x.dtype)
    if _load().oracle_all_gather(x.ctypes.data, out.ctypes.data, P, n, x.dtype.itemsize) != 0:
        raise RuntimeError("oracle_all_gather failed")
    return out


def broadcast(x: np.ndarray, root: int) -> np.ndarray:
    """x[P, n] -> out[P, n]; every rank holds the root's input."""
    _check(x)
    x = np.ascontiguousarray(x)
    P, n = x.shape
    out = np.empty_like(x)
    if _load().oracle_broadcast(x.ctypes.data, out.ctypes.data, P, n, x.dtype.itemsize, root) != 0:
        raise RuntimeError("oracle_broadcast failed")
    return out


def reduce(x: np.ndarray) -> np.ndarray:
    """x[P, n] -> out[n]: the rank-ordered sum (what the root receives)."""
    _check(x)
    x = np.ascontiguousarray(x)
    P, n = x.shape
    out = np.empty(n, dtype=x.dtype)
    if _load().oracle_reduce(x.ctypes.data, out.ctypes.data, P, n, x.dtype.itemsize) != 0:
        raise RuntimeError("oracle_reduce failed")
    return out


def _set_omp_threads(n: int) -> None:
    _load().oracle_set_threads(ctypes.c_int(n))


def narrow_bf16(f: float) -> int:
    return int(_load().oracle_narrow_bf16(ctypes.c_float(f)))


def widen_bf16(h: int) -> float:
    return float(_load().oracle_widen_bf16(ctypes.c_uint16(h)))


# ---------------------------------------------------------------------------
# second reference + error bound (Sec. IV, forward-error bound of summation)
# ---------------------------------------------------------------------------

def bf16_bits_to_f64(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def sum_f64(x: np.ndarray) -> np.ndarray:
    """Elementwise sum over ranks accumulated in binary64 (one row, [count])."""
    kind = _check(x)
    xd = x.astype(np.float64) if kind == "f32" else bf16_bits_to_f64(x)
    return xd.sum(axis=0)


def gamma(k: int, u: float = 2.0 ** -24) -> float:
    """gamma_k = k u / (1 - k u); u defaults to binary32's unit roundoff."""
    return k * u / (1.0 - k * u)


def error_bound(x: np.ndarray, u: float = 2.0 ** -24) -> np.ndarray:
    """gamma_{P-1} * sum_q |x_q| per element, for the binary32 accumulation."""
    kind = _check(x)
    xd = x.astype(np.float64) if kind == "f32" else bf16_bits_to_f64(x)
    return gamma(x.shape[0] - 1, u) * np.abs(xd).sum(axis=0)
