"""The bounds-checking build of the library (libsymar_check.so, -DSYMAR_CHECK): every heap address a
kernel computes is checked against the region it must lie in; a violation is recorded in the status
word and the access skipped.  It stands in for a memory checker where none can be run.

Two things are shown: the checker catches an access outside a call's output range (a self-test whose
stray store stays inside the heap's user region, so it is harmless even unchecked), and the parity
tests -- small and ragged shapes, non-zero offsets, small scratch, every unit width, the bandwidth
kernels, the sibling collectives, the atomic two-shot, one fuzz seed, the static entry point -- run
clean against it: same bits as the oracle and the status word stays SYMAR_OK.  The library is chosen
per process (SYMAR_LIB), so those runs are child processes.
"""
import os
import subprocess
import sys
from pathlib import Path

import pytest

from paper_2607_16100_b200 import build, symar

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def run_with_checking_library(args, timeout):
    lib = build.build_lib_check()
    env = dict(os.environ, SYMAR_LIB=str(lib), PYTHONPATH=str(ROOT))
    return subprocess.run([sys.executable, *args], cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_regular_build_checks_nothing_and_says_so():
    h = symar.SymHeap.on_torch(2, 1 << 16)
    try:
        assert h.check_selftest() == symar.ERR_UNSUPPORTED
        assert h.status()[0] == symar.OK
    finally:
        h.destroy()


def test_checking_build_records_and_skips_an_access_outside_the_output_range():
    code = ("from paper_2607_16100_b200 import symar\n"
            "assert symar.LIB_PATH.name == 'libsymar_check.so'\n"
            "h = symar.SymHeap.on_torch(4, 1 << 16)\n"
            "rc = h.check_selftest()\n"
            "assert rc == symar.OK, rc\n"
            "assert h.status()[0] == symar.OK\n"         # the self-test clears what it provoked
            "print('selftest ok')\n")
    r = run_with_checking_library(["-c", code], 300)
    assert r.returncode == 0 and "selftest ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_parity_tests_run_clean_against_the_checking_build():
    select = ("test_small_shapes or test_nonzero_offsets or test_small_scratch_buffers or test_unit_width_variants "
              "or test_push_many_iterations or test_bandwidth_regime or test_special_values or test_forced_launch_shapes "
              "or test_graph_capture_replays or test_reduce_scatter or test_all_gather or test_broadcast_and_reduce "
              "or test_small_shapes_within_tolerance or (test_random_call_sequences and 8-1) "
              "or test_static_entry_point_matches")
    r = run_with_checking_library(
        ["-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", "-k", select,
         "tests/test_parity_gpu.py", "tests/test_collectives_gpu.py", "tests/test_atomic_gpu.py",
         "tests/test_fuzz_gpu.py", "tests/test_zz_no_alloc.py"], 1500)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout.splitlines()[-1], tail
