"""CPU-side checks of the C-ABI boundary: the library builds, loads without a
GPU, exports every function include/symar.h declares, and its host-only layout
arithmetic matches the sizes the paper's Table I prescribes for LL scratch."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2607_16100_b200 import build, symar

ROOT = Path(__file__).resolve().parent.parent
HEADER = (ROOT / "include" / "symar.h").read_text()


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", HEADER, flags=re.S)
    names = re.findall(r"\b((?:symheap|symar|allreduce)\w*)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    build.build_lib()
    return symar.load()


def test_header_declares_the_three_core_calls():
    names = declared_functions()
    for must in ("symheap_create", "allreduce", "allreduce_autotune"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    raw = ctypes.CDLL(str(symar.LIB_PATH))
    for name in declared_functions():
        assert hasattr(raw, name), f"{name} declared in symar.h but not exported"


def test_binding_covers_every_declared_symbol():
    bound = {n for n, _, _ in symar.SIGNATURES}
    assert bound == set(declared_functions())


def test_binding_constants_match_header():
    for name, val in (("SYMAR_MAX_RANKS", symar.MAX_RANKS), ("SYMAR_MAX_CTAS", symar.MAX_CTAS),
                      ("SYMAR_LL_SLOTS", symar.LL_SLOTS), ("SYMAR_LL_SLOT_VECS", symar.LL_SLOT_VECS),
                      ("SYMAR_ALIGN", symar.ALIGN)):
        m = re.search(rf"{name}\s*=\s*(\d+)", HEADER)
        assert m and int(m.group(1)) == val
    for name, val in (("SYMAR_AUTO", 0), ("SYMAR_ONESHOT", 1), ("SYMAR_TWOSHOT", 2), ("SYMAR_LL", 3),
                      ("SYMAR_SENTINEL", 4), ("SYMAR_TWOSHOT_LL", 5), ("SYMAR_TWOSHOT_SENTINEL", 6),
                      ("SYMAR_TWOSHOT_ATOMIC", 7),
                      ("SYMAR_ERR_TIMEOUT", -4)):
        m = re.search(rf"{name}\s*=\s*(-?\d+)", HEADER)
        assert m and int(m.group(1)) == val


@pytest.mark.parametrize("P", [1, 2, 4, 8])
def test_required_bytes_layout(lib, P):
    user = 1 << 20
    total = symar.required_bytes(P, user)
    # Table I, one-shot LL: scratch per iteration is 2 N D -- every payload byte
    # doubles (flag as large as data) and every rank keeps one row per sender.
    # D here is one slot's payload (vecs x 16 B) times the slots; two parities
    # for double buffering.
    D = symar.LL_SLOTS * symar.LL_SLOT_VECS * 16
    ll = 2 * (2 * P * D)
    # Table I, one-shot sentinel: N D per iteration (bare payload), again two parities
    sentinel = 2 * (P * D)
    # Table I, two-shot LL128 atomic: about D / N per iteration; this build gives every
    # rank two parity halves of 512 KiB x P of 128-byte accumulator lines
    atomic = 2 * (512 << 10) * P
    # flags and counters: two copies of everything, one per half of the chip's L2, in 8 KiB pairs
    # (ready flags 2 pairs, done flags 2 pairs, counters 1 pair)
    flags = 5 * 8192
    assert total >= P * (user + ll + sentinel + atomic + flags)
    assert total <= P * (user + ll + sentinel + atomic + flags + 16 * symar.ALIGN) + 4096
    assert total % symar.ALIGN == 0
    # monotone in the user size, and rounding never loses bytes
    assert symar.required_bytes(P, user + 1) >= total


def test_required_bytes_rejects_bad_rank_counts(lib):
    for P in (0, 3, 5, 16, -1):
        assert symar.required_bytes(P, 4096) == 0


def test_host_side_argument_errors_need_no_gpu(lib):
    h = ctypes.c_void_p()
    assert lib.symheap_create(ctypes.byref(h), 3, 4096) == symar.ERR_INVAL
    assert lib.symheap_create(None, 4, 4096) == symar.ERR_INVAL
    assert lib.symheap_create(ctypes.byref(h), 4, 0) == symar.ERR_INVAL
    assert lib.symheap_destroy(None) == symar.ERR_INVAL
    assert lib.allreduce(None, None, None, 0, 0, 0, None) == symar.ERR_INVAL
    assert lib.symar_probe_empty(0, 1, 32, None) == symar.ERR_INVAL
