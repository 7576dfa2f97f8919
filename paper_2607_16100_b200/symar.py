"""ctypes binding of libsymar.so: argument marshalling only.

Function names and argument order follow ``include/symar.h``.  Every step of
the collective runs in the library's CUDA kernels; if the library is missing
or fails to load this module raises -- there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_int, c_size_t, c_uint, c_void_p
from pathlib import Path

_PKG = Path(__file__).resolve().parent
# SYMAR_LIB selects another build of the same library (the system-scope or the bounds-checking
# flavour of paper_2607_16100_b200/build.py); by default the regular one.
LIB_PATH = Path(os.environ["SYMAR_LIB"]) if os.environ.get("SYMAR_LIB") else _PKG / "libsymar.so"

F32, BF16 = 0, 1
AUTO, ONESHOT, TWOSHOT, LL, SENTINEL, TWOSHOT_LL, TWOSHOT_SENTINEL, TWOSHOT_ATOMIC = 0, 1, 2, 3, 4, 5, 6, 7
ALGO_NAMES = {AUTO: "auto", ONESHOT: "oneshot", TWOSHOT: "twoshot", LL: "ll", SENTINEL: "sentinel",
              TWOSHOT_LL: "twoshot_ll", TWOSHOT_SENTINEL: "twoshot_sentinel", TWOSHOT_ATOMIC: "twoshot_atomic"}
DTYPE_NAMES = {F32: "f32", BF16: "bf16"}
DTYPE_SIZE = {F32: 4, BF16: 2}

OK, ERR_INVAL, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5
_ERR_NAMES = {
    ERR_INVAL: "SYMAR_ERR_INVAL", ERR_NOMEM: "SYMAR_ERR_NOMEM", ERR_CUDA: "SYMAR_ERR_CUDA",
    ERR_TIMEOUT: "SYMAR_ERR_TIMEOUT", ERR_UNSUPPORTED: "SYMAR_ERR_UNSUPPORTED",
}

MAX_RANKS, MAX_CTAS, LL_SLOTS, LL_SLOT_VECS, ALIGN = 8, 160, 64, 1024, 8192
VARIANT_CLUSTER = 0x40000000      # SYMAR_VARIANT_CLUSTER: the ranks of a slot launched as one thread-block cluster

# every symbol include/symar.h declares: (name, restype, argtypes)
SIGNATURES = [
    ("symheap_required_bytes", c_size_t, [c_int, c_size_t]),
    ("symheap_create", c_int, [POINTER(c_void_p), c_int, c_size_t]),
    ("symheap_create_on", c_int, [POINTER(c_void_p), c_int, c_size_t, c_void_p, c_size_t]),
    ("symheap_destroy", c_int, [c_void_p]),
    ("symheap_info", c_int, [c_void_p, c_void_p]),
    ("symheap_rank_ptr", c_void_p, [c_void_p, c_int, c_size_t]),
    ("symheap_reset", c_int, [c_void_p, c_void_p]),
    ("symheap_status", c_int, [c_void_p, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_int)]),
    ("allreduce", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int, c_void_p]),
    ("allreduce_host", c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int,
                               c_void_p]),
    ("symar_reduce_scatter", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_void_p]),
    ("symar_all_gather", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_void_p]),
    ("symar_broadcast", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int, c_void_p]),
    ("symar_reduce", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int, c_void_p]),
    ("allreduce_autotune", c_int, [c_void_p, c_int]),
    ("allreduce_autotune_size", c_int, [c_void_p, c_int, c_size_t]),
    ("allreduce_autotune_stream", c_int, [c_void_p, c_int, c_size_t, c_int]),
    ("symar_last_choice", c_int, [c_void_p, POINTER(c_int), POINTER(c_int), POINTER(c_int)]),
    ("symar_last_kernel", c_int, [c_void_p, POINTER(c_uint), POINTER(c_size_t)]),
    ("symar_query_choice", c_int, [c_void_p, c_size_t, c_int, POINTER(c_int), POINTER(c_int), POINTER(c_int)]),
    ("symar_tuned_entry", c_int, [c_void_p, c_int, c_int, c_int, POINTER(c_int), POINTER(c_int),
                                  POINTER(c_double)]),
    ("symar_table_save", c_int, [c_void_p, c_char_p]),
    ("symar_table_load", c_int, [c_void_p, c_char_p]),
    ("symar_set_launch", c_int, [c_void_p, c_int, c_int, c_int]),
    ("symar_set_variant", c_int, [c_void_p, c_int, c_uint]),
    ("symar_set_pdl", c_int, [c_void_p, c_int]),
    ("symar_set_placement", c_int, [c_void_p, c_int]),
    ("symar_placement", c_int, [c_void_p, POINTER(c_int), POINTER(c_int), POINTER(ctypes.c_ulonglong)]),
    ("symar_set_scratch_limit", c_int, [c_void_p, c_size_t]),
    ("symar_set_spin_limit_us", c_int, [c_void_p, c_uint]),
    ("symar_debug_inject", c_int, [c_void_p, c_int, c_uint, c_uint]),
    ("allreduce_static", c_int, [c_void_p, c_void_p, c_size_t, c_int, c_size_t, c_int, c_void_p, c_void_p]),
    ("symar_last_cuda_error", c_char_p, []),
    ("symar_probe_empty", c_int, [c_int, c_int, c_int, c_void_p]),
    ("symar_probe_empty_pdl", c_int, [c_int, c_int, c_int, c_void_p]),
    ("symar_probe_empty_cluster", c_int, [c_int, c_int, c_int, c_void_p]),
    ("symar_probe_fence", c_int, [c_int, POINTER(c_double)]),
    ("symar_probe_pingpong", c_int, [c_int, POINTER(c_double)]),
    ("symar_probe_pingpong_pair", c_int, [c_int, c_int, POINTER(c_double), POINTER(c_int)]),
    ("symar_debug_span", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int, c_void_p, POINTER(c_double)]),
    ("symar_debug_phases", c_int, [c_void_p, c_void_p, c_void_p, c_size_t, c_int, c_int, c_void_p, POINTER(c_double),
                                   POINTER(c_int)]),
    ("symar_check_selftest", c_int, [c_void_p, c_void_p]),
    ("symar_probe_barrier", c_int, [c_int, c_int, c_int, POINTER(c_double)]),
    ("symar_llbuffer_bytes", c_size_t, [c_int, c_size_t, c_size_t, c_int, c_int]),
    ("symar_llbuffer_init_sentinel", c_int, [c_void_p, c_size_t, c_void_p]),
    ("symar_probe_pingpong_blocks", c_int, [c_int, c_int, c_int, c_int, POINTER(c_double), POINTER(c_int)]),
]


class SymarError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code == ERR_CUDA and _lib is not None:
            detail = ": " + (_lib.symar_last_cuda_error() or b"").decode()
        super().__init__(f"{where} -> {_ERR_NAMES.get(code, code)}{detail}")


class HeapInfo(ctypes.Structure):
    _fields_ = [
        ("P", c_int), ("bytes_per_rank", c_size_t), ("user_bytes", c_size_t),
        ("ll_scratch_bytes", c_size_t), ("sentinel_scratch_bytes", c_size_t), ("atomic_scratch_bytes", c_size_t),
        ("flag_bytes", c_size_t),
        ("stride", c_size_t),
        ("total_bytes", c_size_t), ("base", c_void_p),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """dlopen the library and declare every signature.  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(
                f"{LIB_PATH} not found: build it with `python -m paper_2607_16100_b200.build` "
                "(there is no non-CUDA path)")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, res, args in SIGNATURES:
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ck(rc: int, where: str) -> None:
    if rc != OK:
        raise SymarError(rc, where)


def required_bytes(P: int, bytes_per_rank: int) -> int:
    return int(load().symheap_required_bytes(P, bytes_per_rank))


class SymHeap:
    """Owner of one ``symheap_t``.  ``device_mem`` (an int address) + ``device_bytes``
    place the heap in caller memory (``symheap_create_on``); otherwise the library
    allocates (``symheap_create``)."""

    def __init__(self, P: int, bytes_per_rank: int, device_mem: int | None = None,
                 device_bytes: int = 0, keepalive=None):
        self._lib = load()
        self._h = c_void_p()
        self._keepalive = keepalive
        if device_mem is None:
            _ck(self._lib.symheap_create(byref(self._h), P, bytes_per_rank), "symheap_create")
        else:
            _ck(self._lib.symheap_create_on(byref(self._h), P, bytes_per_rank, device_mem, device_bytes),
                "symheap_create_on")
        self.P = P
        self.bytes_per_rank = bytes_per_rank
        i = self.info()
        self.base = int(i.base)
        self.stride = int(i.stride)

    @classmethod
    def on_torch(cls, P: int, bytes_per_rank: int, device="cuda:0") -> "SymHeap":
        """Heap in a torch uint8 tensor (PyTorch provides the device memory)."""
        import torch
        n = required_bytes(P, bytes_per_rank)
        buf = torch.empty(n + ALIGN, dtype=torch.uint8, device=device)
        addr = (buf.data_ptr() + ALIGN - 1) // ALIGN * ALIGN
        with torch.cuda.device(buf.device):
            return cls(P, bytes_per_rank, addr, n, keepalive=buf)

    # -- lifetime --
    def destroy(self) -> None:
        if self._h:
            self._lib.symheap_destroy(self._h)
            self._h = c_void_p()
            self._keepalive = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- layout --
    def info(self) -> HeapInfo:
        i = HeapInfo()
        _ck(self._lib.symheap_info(self._h, byref(i)), "symheap_info")
        return i

    def rank_ptr(self, rank: int, offset: int = 0) -> int:
        p = self._lib.symheap_rank_ptr(self._h, rank, offset)
        if not p:
            raise SymarError(ERR_INVAL, "symheap_rank_ptr")
        return int(p)

    def reset(self, stream: int = 0) -> None:
        _ck(self._lib.symheap_reset(self._h, stream), "symheap_reset")

    def status(self):
        code, rank, peer, cta = c_int(), c_int(), c_int(), c_int()
        _ck(self._lib.symheap_status(self._h, byref(code), byref(rank), byref(peer), byref(cta)),
            "symheap_status")
        return code.value, rank.value, peer.value, cta.value

    # -- the collective --
    def allreduce_rc(self, in_off: int, out_off: int, count: int, dtype: int, algo: int = AUTO,
                     stream: int = 0) -> int:
        """Raw status code; offsets are turned into rank-0 symmetric addresses."""
        base = self.base
        return int(self._lib.allreduce(self._h, base + in_off, base + out_off, count, dtype, algo, stream))

    def allreduce(self, in_off: int, out_off: int, count: int, dtype: int, algo: int = AUTO,
                  stream: int = 0) -> None:
        _ck(self.allreduce_rc(in_off, out_off, count, dtype, algo, stream), "allreduce")

    def allreduce_ptr(self, in_ptr: int, out_ptr: int, count: int, dtype: int, algo: int = AUTO,
                      stream: int = 0) -> None:
        _ck(self._lib.allreduce(self._h, in_ptr, out_ptr, count, dtype, algo, stream), "allreduce")

    def allreduce_host(self, host_in: int, host_out: int, in_off: int, out_off: int, count: int,
                       dtype: int, algo: int = AUTO, stream: int = 0) -> None:
        base = self.base
        _ck(self._lib.allreduce_host(self._h, host_in, host_out, base + in_off, base + out_off, count,
                                     dtype, algo, stream), "allreduce_host")

    # -- sibling collectives (raw status codes; offsets become rank-0 symmetric addresses) --
    def reduce_scatter(self, in_off, out_off, recv_count, dtype, stream=0) -> int:
        return int(self._lib.symar_reduce_scatter(self._h, self.base + in_off, self.base + out_off, recv_count,
                                                  dtype, stream))

    def all_gather(self, in_off, out_off, send_count, dtype, stream=0) -> int:
        return int(self._lib.symar_all_gather(self._h, self.base + in_off, self.base + out_off, send_count,
                                              dtype, stream))

    def broadcast(self, in_off, out_off, count, dtype, root, stream=0) -> int:
        return int(self._lib.symar_broadcast(self._h, self.base + in_off, self.base + out_off, count, dtype,
                                             root, stream))

    def reduce(self, in_off, out_off, count, dtype, root, stream=0) -> int:
        return int(self._lib.symar_reduce(self._h, self.base + in_off, self.base + out_off, count, dtype, root,
                                          stream))

    # -- data movement helpers for heaps that live in a torch tensor --
    def _bytes_view(self, rank: int, offset: int, nbytes: int):
        if self._keepalive is None:
            raise RuntimeError("heap does not live in a torch tensor (use SymHeap.on_torch)")
        if not (0 <= rank < self.P) or offset < 0 or offset + nbytes > self.bytes_per_rank:
            raise SymarError(ERR_INVAL, "rank/offset/size outside the user region")
        start = self.base + rank * self.stride + offset - self._keepalive.data_ptr()
        return self._keepalive[start:start + nbytes]

    def write_rank(self, rank: int, offset: int, array) -> None:
        """Copy a host numpy array into rank ``rank``'s user region at ``offset``."""
        import numpy as np
        import torch
        a = np.ascontiguousarray(array)
        src = torch.from_numpy(a.view(np.uint8).reshape(-1))
        self._bytes_view(rank, offset, a.nbytes).copy_(src, non_blocking=False)

    def read_rank(self, rank: int, offset: int, count: int, np_dtype):
        """Copy ``count`` elements of ``np_dtype`` from rank ``rank``'s user region to the host."""
        import numpy as np
        n = count * np.dtype(np_dtype).itemsize
        return self._bytes_view(rank, offset, n).cpu().numpy().view(np_dtype).copy()

    def fill_user(self, byte: int) -> None:
        """Fill every rank's user region with one byte value (poison before a test)."""
        for q in range(self.P):
            self._bytes_view(q, 0, self.bytes_per_rank).fill_(byte)

    # -- selector --
    def autotune(self, dtype: int) -> None:
        _ck(self._lib.allreduce_autotune(self._h, dtype), "allreduce_autotune")

    def autotune_size(self, dtype: int, count: int) -> None:
        _ck(self._lib.allreduce_autotune_size(self._h, dtype, count), "allreduce_autotune_size")

    def autotune_stream(self, dtype: int, count: int, calls: int) -> None:
        _ck(self._lib.allreduce_autotune_stream(self._h, dtype, count, calls), "allreduce_autotune_stream")

    def last_choice(self):
        a, c, t = c_int(), c_int(), c_int()
        _ck(self._lib.symar_last_choice(self._h, byref(a), byref(c), byref(t)), "symar_last_choice")
        return a.value, c.value, t.value

    def last_kernel(self):
        v, sm = c_uint(), c_size_t()
        _ck(self._lib.symar_last_kernel(self._h, byref(v), byref(sm)), "symar_last_kernel")
        return v.value, sm.value

    def query_choice(self, count: int, dtype: int, algo: int = AUTO):
        a, c, t = c_int(algo), c_int(), c_int()
        _ck(self._lib.symar_query_choice(self._h, count, dtype, byref(a), byref(c), byref(t)),
            "symar_query_choice")
        return a.value, c.value, t.value

    def tuned_entry(self, dtype: int, log2_bytes: int, algo: int):
        c, t, us = c_int(), c_int(), c_double()
        rc = self._lib.symar_tuned_entry(self._h, dtype, log2_bytes, algo, byref(c), byref(t), byref(us))
        if rc != OK:
            return None
        return c.value, t.value, us.value

    def table_save(self, path: str) -> None:
        _ck(self._lib.symar_table_save(self._h, str(path).encode()), "symar_table_save")

    def table_load(self, path: str) -> None:
        _ck(self._lib.symar_table_load(self._h, str(path).encode()), "symar_table_load")

    def set_launch(self, algo: int, ctas_per_rank: int, threads: int) -> None:
        _ck(self._lib.symar_set_launch(self._h, algo, ctas_per_rank, threads), "symar_set_launch")

    def set_variant(self, algo: int, variant: int) -> None:
        _ck(self._lib.symar_set_variant(self._h, algo, variant), "symar_set_variant")

    def set_pdl(self, enabled: bool) -> None:
        _ck(self._lib.symar_set_pdl(self._h, 1 if enabled else 0), "symar_set_pdl")

    def set_placement(self, enabled: bool) -> None:
        _ck(self._lib.symar_set_placement(self._h, 1 if enabled else 0), "symar_set_placement")

    def placement(self):
        """(measured cleanly?, SMs on the second L2 half, home bits)"""
        m, n, hb = c_int(), c_int(), ctypes.c_ulonglong()
        _ck(self._lib.symar_placement(self._h, byref(m), byref(n), byref(hb)), "symar_placement")
        return bool(m.value), n.value, hb.value

    def set_scratch_limit(self, payload_bytes_per_iteration: int) -> None:
        _ck(self._lib.symar_set_scratch_limit(self._h, payload_bytes_per_iteration), "symar_set_scratch_limit")

    def set_spin_limit_us(self, us: int) -> None:
        _ck(self._lib.symar_set_spin_limit_us(self._h, us), "symar_set_spin_limit_us")

    def debug_span(self, in_off: int, out_off: int, count: int, dtype: int, algo: int = AUTO, stream: int = 0) -> float:
        """In-kernel span in ns (first CTA in -> last CTA out) of one synchronous call."""
        v = c_double()
        _ck(self._lib.symar_debug_span(self._h, self.rank_ptr(0, in_off), self.rank_ptr(0, out_off), count, dtype,
                                       algo, stream, byref(v)), "symar_debug_span")
        return v.value

    def debug_phases(self, in_off: int, out_off: int, count: int, dtype: int, algo: int = AUTO, stream: int = 0):
        """Per phase k = 0..7 of one synchronous call: (earliest, mean, latest) ns since the first CTA's
        start, and how many CTAs stamped it; phases the kernel does not have are left out."""
        ns = (c_double * 24)()
        n = (c_int * 8)()
        _ck(self._lib.symar_debug_phases(self._h, self.rank_ptr(0, in_off), self.rank_ptr(0, out_off), count, dtype,
                                         algo, stream, ns, n), "symar_debug_phases")
        return {k: {"first": ns[3 * k], "mean": ns[3 * k + 1], "last": ns[3 * k + 2], "ctas": n[k]}
                for k in range(8) if n[k] > 0}

    def check_selftest(self, stream: int = 0) -> int:
        """Raw status of the bounds-checking build's self-test (ERR_UNSUPPORTED in the regular build)."""
        return int(self._lib.symar_check_selftest(self._h, stream))

    def debug_inject(self, mute_rank: int = -1, delay_seed: int = 0, delay_max_ns: int = 0) -> None:
        _ck(self._lib.symar_debug_inject(self._h, mute_rank, delay_seed, delay_max_ns), "symar_debug_inject")


STATIC_MAX_BYTES = 32768


def allreduce_static(in_ptr: int, out_ptr: int, rank_pitch_bytes: int, P: int, count: int, dtype: int,
                     status_ptr: int = 0, stream: int = 0) -> int:
    """AllReduce on plain device buffers with library-internal static scratch; the
    library allocates nothing.  Returns the raw status code."""
    return int(load().allreduce_static(in_ptr, out_ptr, rank_pitch_bytes, P, count, dtype,
                                       status_ptr or None, stream))


# -- probes --

def probe_empty(grid_x: int, grid_y: int, block: int, stream: int = 0) -> None:
    _ck(load().symar_probe_empty(grid_x, grid_y, block, stream), "symar_probe_empty")


def probe_empty_pdl(grid_x: int, grid_y: int, block: int, stream: int = 0) -> None:
    _ck(load().symar_probe_empty_pdl(grid_x, grid_y, block, stream), "symar_probe_empty_pdl")


def probe_empty_cluster(grid_x: int, grid_y: int, block: int, stream: int = 0) -> None:
    _ck(load().symar_probe_empty_cluster(grid_x, grid_y, block, stream), "symar_probe_empty_cluster")


def probe_fence(iterations: int = 20000) -> float:
    v = c_double()
    _ck(load().symar_probe_fence(iterations, byref(v)), "symar_probe_fence")
    return v.value


def probe_pingpong(iterations: int = 20000) -> float:
    v = c_double()
    _ck(load().symar_probe_pingpong(iterations, byref(v)), "symar_probe_pingpong")
    return v.value


def llbuffer_bytes(sync_mode: int, elem_bytes: int, slots_per_cta: int, ctas: int, round_robin: int) -> int:
    return int(load().symar_llbuffer_bytes(sync_mode, elem_bytes, slots_per_cta, ctas, round_robin))


def llbuffer_init_sentinel(device_ptr: int, nbytes: int, stream: int = 0) -> None:
    _ck(load().symar_llbuffer_init_sentinel(device_ptr, nbytes, stream), "symar_llbuffer_init_sentinel")


def probe_barrier(ranks: int, iterations: int = 5000, ordered: bool = False) -> float:
    """ns per all-to-all flag barrier among `ranks` CTAs (the barrier the method removes)."""
    v = c_double()
    _ck(load().symar_probe_barrier(ranks, iterations, 1 if ordered else 0, byref(v)), "symar_probe_barrier")
    return v.value


def probe_pingpong_blocks(first_block: int, partner_block: int, grid_blocks: int, iterations: int = 20000):
    """(ns per round trip, (smid_first, smid_partner)); only the two named blocks of the launch play."""
    v = c_double()
    sm = (c_int * 2)()
    _ck(load().symar_probe_pingpong_blocks(iterations, first_block, partner_block, grid_blocks, byref(v), sm),
        "symar_probe_pingpong_blocks")
    return v.value, (sm[0], sm[1])


def probe_pingpong_pair(partner_block: int, iterations: int = 20000):
    """(ns per round trip, (smid0, smid1)) between block 0 and block `partner_block`."""
    v = c_double()
    sm = (c_int * 2)()
    _ck(load().symar_probe_pingpong_pair(iterations, partner_block, byref(v), sm), "symar_probe_pingpong_pair")
    return v.value, (sm[0], sm[1])
