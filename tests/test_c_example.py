"""The library from a plain C program (examples/allreduce_from_c.c): the header compiles as C99 with gcc
alone (CPU), and the program's result equals the oracle's bit for bit (GPU)."""
import subprocess

import numpy as np
import pytest

from paper_2607_16100_b200 import build, synth


def test_header_is_plain_c_and_the_program_links():
    exe = build.build_c_example(force=True)          # gcc -std=c99 -pedantic -Wall -Wextra -Werror
    assert exe.exists()
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 2 and "usage" in r.stderr


@pytest.mark.gpu
@pytest.mark.parametrize("P,dtype,count,algo", [
    (8, "bf16", 8192, 0),            # AUTO at the decode-step message
    (4, "f32", 1024, 1),             # the smallest workload: one-shot
    (8, "f32", 300001, 2),           # two-shot, ragged
    (2, "bf16", 777, 3),             # the data+flag protocol
    (8, "f32", 9 * (1 << 20) + 5, 0),    # 36 MiB per rank: the chunked host pipeline from pageable memory
])
def test_c_program_matches_the_oracle(tmp_path, P, dtype, count, algo):
    from oracle import allreduce_oracle as O
    exe = build.build_c_example()
    x = synth.make_inputs("uniform" if dtype == "f32" else "normal", dtype, P, count, seed=4000 + count)
    fin, fout = tmp_path / "in.bin", tmp_path / "out.bin"
    x.tofile(fin)
    r = subprocess.run([str(exe), str(P), "0" if dtype == "f32" else "1", str(count), str(algo), str(fin), str(fout)],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    got = np.fromfile(fout, dtype=x.dtype).reshape(P, count)
    want = O.allreduce(x)
    bits = np.uint32 if dtype == "f32" else np.uint16
    assert np.array_equal(got.view(bits), want.view(bits)), r.stdout
