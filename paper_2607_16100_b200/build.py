"""Build libsymar.so (the C-ABI CUDA library) and the example kernel written on the public
device header, in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libsymar.so"
SOURCES = ["symar_kernels.cu", "symar_bulk.cu", "symar_host.cu", "symar_probe.cu", "symar_static.cu", "symar_coll.cu",
           "symar_atomic.cu", "symar_place.cu"]

LIB_SYS = PKG / "libsymar_sys.so"
LIB_CHECK = PKG / "libsymar_check.so"

EXAMPLE_SRC = PKG / "examples" / "llbuffer_oneshot.cu"
EXAMPLE_LIB = PKG / "libsymar_example.so"
C_EXAMPLE_SRC = PKG / "examples" / "allreduce_from_c.c"
C_EXAMPLE_BIN = PKG / "allreduce_from_c.bin"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true", "--fmad=false",
    "-cudart", "static",
    "--threads", "0",
]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.iterdir()) + [ROOT / "include" / "symar.h", Path(__file__)]   # (the example has its own check)
    return any(d.stat().st_mtime > t for d in deps)


def build_lib(force: bool = False, verbose: bool = False) -> Path:
    """Compile the library if a source is newer than it.  Needs nvcc only (no GPU)."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, *NVCC_FLAGS, "-I", str(ROOT / "include"), "-I", str(CSRC),
           "-o", str(tmp), *[str(CSRC / s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


def _build_flavour(lib: Path, define: str, force: bool) -> Path:
    deps = list(CSRC.iterdir()) + [ROOT / "include" / "symar.h", Path(__file__)]
    if not force and lib.exists() and all(d.stat().st_mtime <= lib.stat().st_mtime for d in deps):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, *NVCC_FLAGS, define, "-I", str(ROOT / "include"), "-I", str(CSRC),
           "-o", str(tmp), *[str(CSRC / s) for s in SOURCES]]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


def build_lib_sys(force: bool = False) -> Path:
    """The same library with every flag, signal and data+flag access at SYSTEM scope (what ranks on
    several GPUs of one NVLink domain need), for timing beside the default.  Load it by setting
    SYMAR_LIB to its path before importing the binding."""
    return _build_flavour(LIB_SYS, "-DSYMAR_SCOPE_SYS", force)


def build_lib_check(force: bool = False) -> Path:
    """The bounds-checking debug build: every heap address a kernel computes is checked against the
    region it must lie in before it is used; a violation records SYMAR_ERR_INVAL with the rank, the
    CTA slot and the region in the status word and skips the access.  Slower; for tests.  Load it by
    setting SYMAR_LIB to its path before importing the binding."""
    return _build_flavour(LIB_CHECK, "-DSYMAR_CHECK", force)


def build_example(force: bool = False) -> Path:
    """The one-shot AllReduce of examples/llbuffer_oneshot.cu: uses include/symar_llbuffer.cuh only."""
    deps = [EXAMPLE_SRC, ROOT / "include" / "symar_llbuffer.cuh", Path(__file__)]
    if not force and EXAMPLE_LIB.exists() and all(d.stat().st_mtime <= EXAMPLE_LIB.stat().st_mtime for d in deps):
        return EXAMPLE_LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = EXAMPLE_LIB.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, *NVCC_FLAGS, "--extended-lambda", "-I", str(ROOT / "include"), "-o", str(tmp), str(EXAMPLE_SRC)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, EXAMPLE_LIB)
    return EXAMPLE_LIB


def build_c_example(force: bool = False) -> Path:
    """examples/allreduce_from_c.c: a plain C99 program on include/symar.h and libsymar.so alone (gcc, no
    CUDA header); also the check that the header is valid C."""
    build_lib()
    deps = [C_EXAMPLE_SRC, ROOT / "include" / "symar.h", LIB, Path(__file__)]
    if not force and C_EXAMPLE_BIN.exists() and all(d.stat().st_mtime <= C_EXAMPLE_BIN.stat().st_mtime for d in deps):
        return C_EXAMPLE_BIN
    tmp = C_EXAMPLE_BIN.with_suffix(f".bin.tmp{os.getpid()}")
    cmd = [os.environ.get("CC", "gcc"), "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-O2",
           "-I", str(ROOT / "include"), str(C_EXAMPLE_SRC), "-L", str(PKG), "-lsymar", "-Wl,-rpath,$ORIGIN",
           "-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, C_EXAMPLE_BIN)
    return C_EXAMPLE_BIN


if __name__ == "__main__":
    print(build_lib(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_example(force="--force" in sys.argv))
    print(build_c_example(force="--force" in sys.argv))
    if "--sys" in sys.argv:
        print(build_lib_sys(force="--force" in sys.argv))
    if "--check" in sys.argv:
        print(build_lib_check(force="--force" in sys.argv))
