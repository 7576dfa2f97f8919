"""Seeded random sequences of calls on ONE heap: every algorithm, both dtypes, ragged counts, random
offsets, forced launch shapes, kernel variants, limited scratch, with and without programmatic dependent
launch, the sibling collectives in between, batches enqueued without host synchronisation.  All state
that survives a call (flags, per-slot counters, scratch parity, sentinels, accumulator lines) must stay
consistent whatever the order.  Every result is compared with the oracle: bit for bit, except for the
atomic two-shot (tolerance, and identical bits on all ranks)."""
import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import symar, synth

pytestmark = pytest.mark.gpu

USER = 4 << 20
NP_DT = {symar.F32: np.float32, symar.BF16: np.uint16}
NAME = {symar.F32: "f32", symar.BF16: "bf16"}
EXACT = [symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL,
         symar.AUTO]


def widen(a):
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def check_atomic(got, x, want, what):
    for q in range(1, got.shape[0]):
        assert np.array_equal(got[q], got[0]), f"{what}: rank {q} differs"
    g, w = widen(got[0]), widen(want[0])
    tol = 1e-6 * np.abs(widen(x)).sum(axis=0)
    if got.dtype == np.uint16:
        tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(w), 1e-30))) - 7)
    assert np.all(np.abs(g - w) <= tol), what


@pytest.mark.parametrize("P,seed", [(8, 1), (4, 2), (2, 3), (8, 4), (1, 5)])
def test_random_call_sequences(P, seed):
    rng = np.random.default_rng(seed)
    h = symar.SymHeap.on_torch(P, USER)
    try:
        pending = []                                   # calls enqueued but not yet checked

        def flush():
            torch.cuda.synchronize()
            assert h.status()[0] == symar.OK, f"device status {h.status()}"
            for kind, out_off, n_out, dt, x, want, what in pending:
                got = np.stack([h.read_rank(q, out_off, n_out, NP_DT[dt]) for q in range(P)])
                if kind == "atomic":
                    check_atomic(got, x, want, what)
                elif kind == "reduce":                 # only the root's output is defined
                    root, w = want
                    assert np.array_equal(got[root].view(np.uint8), w.view(np.uint8)), what
                else:
                    assert np.array_equal(got.view(np.uint8), want.view(np.uint8)), what
            pending.clear()

        regions = [(i * (USER // 8), USER // 8) for i in range(8)]     # 8 disjoint 512 KiB regions
        for step in range(140):
            dt = symar.BF16 if rng.random() < 0.5 else symar.F32
            es = 2 if dt == symar.BF16 else 4
            big = rng.random() < 0.15
            count = int(rng.integers(1, (USER // 8) // es if big else 6000))
            ri, ro = rng.choice(8, size=2, replace=False)
            in_off = regions[ri][0] + 16 * int(rng.integers(0, 4))
            out_off = regions[ro][0] + 16 * int(rng.integers(0, 4))
            count = min(count, (USER // 8 - 64) // es)
            # a region may not be reused while a pending call still reads or writes it
            if any(p_[1] // (USER // 8) in (ri, ro) for p_ in pending) or len(pending) >= 4 or rng.random() < 0.3:
                flush()
            r = rng.random()
            what = f"P={P} seed={seed} step={step}"
            if r < 0.78:
                algo = int(rng.choice(EXACT + [symar.TWOSHOT_ATOMIC]))
                if rng.random() < 0.3 and algo != symar.AUTO:
                    h.set_launch(algo, int(rng.choice([1, 2, 3, 5, 8, 16, 40])), int(rng.choice([32, 64, 96, 128, 256, 512])))
                if rng.random() < 0.3 and algo != symar.AUTO:
                    # unit widths, the plain form, each slot's ranks as a cluster or not (whatever the built-in rule says)
                    cl = symar.VARIANT_CLUSTER
                    choices = {symar.ONESHOT: [0x100, 0x200, 1 << 31, cl, cl | 0x100],
                               symar.LL: [0x100, 1 << 31, cl | 0x100, cl | 0x2100, cl | 0x200],
                               symar.TWOSHOT: [0x40, 1 << 31, cl, cl | 0x40]}.get(algo, [1 << 31, cl])
                    h.set_variant(algo, int(rng.choice(choices)))
                if rng.random() < 0.15:
                    h.set_scratch_limit(int(rng.choice([0, 4096, 65536])))
                if rng.random() < 0.2:
                    h.set_pdl(bool(rng.random() < 0.5))
                x = synth.make_inputs("normal" if dt == symar.BF16 else "uniform", NAME[dt], P, count, seed=seed * 1000 + step)
                for q in range(P):
                    h.write_rank(q, in_off, x[q])
                if algo == symar.TWOSHOT_ATOMIC and count > 31 * 4096 * P * P:
                    # beyond what one call of the atomic two-shot can reduce: refused, nothing launched
                    assert h.allreduce_rc(in_off, out_off, count, dt, algo) == symar.ERR_UNSUPPORTED, what
                    continue
                h.allreduce(in_off, out_off, count, dt, algo)
                pending.append(("atomic" if algo == symar.TWOSHOT_ATOMIC else "exact", out_off, count, dt, x,
                                O.allreduce(x), what + f" algo={algo} count={count}"))
                if algo != symar.AUTO:
                    h.set_launch(algo, 0, 0)
                    h.set_variant(algo, 0)
            else:
                n = max(1, count // P)
                op = int(rng.integers(0, 4))
                root = int(rng.integers(0, P))
                if op == 0:
                    x = synth.make_inputs("uniform", NAME[dt], P, n * P, seed=step)
                    for q in range(P):
                        h.write_rank(q, in_off, x[q])
                    assert h.reduce_scatter(in_off, out_off, n, dt) == symar.OK
                    pending.append(("exact", out_off, n, dt, x, O.reduce_scatter(x), what + " reduce_scatter"))
                elif op == 1:
                    x = synth.make_inputs("uniform", NAME[dt], P, n, seed=step)
                    for q in range(P):
                        h.write_rank(q, in_off, x[q])
                    assert h.all_gather(in_off, out_off, n, dt) == symar.OK
                    pending.append(("exact", out_off, n * P, dt, x, O.all_gather(x), what + " all_gather"))
                elif op == 2:
                    x = synth.make_inputs("uniform", NAME[dt], P, n, seed=step)
                    for q in range(P):
                        h.write_rank(q, in_off, x[q])
                    assert h.broadcast(in_off, out_off, n, dt, root) == symar.OK
                    pending.append(("exact", out_off, n, dt, x, O.broadcast(x, root), what + " broadcast"))
                else:
                    x = synth.make_inputs("uniform", NAME[dt], P, n, seed=step)
                    for q in range(P):
                        h.write_rank(q, in_off, x[q])
                    assert h.reduce(in_off, out_off, n, dt, root) == symar.OK
                    pending.append(("reduce", out_off, n, dt, x, (root, O.reduce(x)), what + " reduce"))
        flush()
        h.set_scratch_limit(0)
        h.set_pdl(True)
    finally:
        torch.cuda.synchronize()
        h.destroy()
