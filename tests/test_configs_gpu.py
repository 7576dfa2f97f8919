"""The five benchmark workloads at their full sizes, in the launch configuration
bench.py times, bit for bit against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import symar, synth

pytestmark = pytest.mark.gpu

ALGOS = [symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL,
         symar.AUTO]
DT = {"f32": symar.F32, "bf16": symar.BF16}
NP = {"f32": np.float32, "bf16": np.uint16}


def bits(a):
    return np.ascontiguousarray(a).view(np.uint8)


def one_call(h, x, dtype, algo, in_off, out_off):
    P, count = x.shape
    for q in range(P):
        h.write_rank(q, in_off, x[q])
    h.allreduce(in_off, out_off, count, DT[dtype], algo)
    torch.cuda.synchronize()
    assert h.status()[0] == symar.OK
    return np.stack([h.read_rank(q, out_off, count, NP[dtype]) for q in range(P)])


def test_c1_exact_integer_sums_p4_fp32():
    w = synth.WORKLOADS["c1"]
    x = synth.make_inputs(w["dist"], w["dtype"], w["P"], w["count"], w["seed"])
    want = O.allreduce(x)
    assert np.array_equal(want[0], x.astype(np.int64).sum(axis=0).astype(np.float32))   # the config's own point
    h = symar.SymHeap.on_torch(w["P"], 1 << 20)
    try:
        for algo in ALGOS:
            got = one_call(h, x, "f32", algo, 0, 1 << 19)
            assert np.array_equal(bits(got), bits(want)), algo
    finally:
        h.destroy()


def test_c2_and_c3_message_sweep_p8_bf16():
    w = synth.WORKLOADS["c3"]
    h = symar.SymHeap.on_torch(8, 4 << 20)
    try:
        for tuned in (False, True):
            if tuned:
                h.autotune(symar.BF16)
            for B in w["batch"]:
                count = w["count"] * B
                x = synth.make_inputs(w["dist"], "bf16", 8, count, w["seed"] + B)
                want = O.allreduce(x)
                for algo in ALGOS:
                    got = one_call(h, x, "bf16", algo, 0, 2 << 20)
                    assert np.array_equal(bits(got), bits(want)), (tuned, B, algo)
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_pruned_tuner_is_quick_and_finds_what_the_exhaustive_search_finds(monkeypatch):
    # The tuner skips algorithms that lost clearly one size down and searches shapes around the previous
    # winner.  It must stay within seconds, and at every c3 size its choice must be as fast as the best
    # entry of a search that prunes nothing (each tuner's own timings; 8 % covers their run-to-run noise).
    import time
    w = synth.WORKLOADS["c3"]
    h = symar.SymHeap.on_torch(8, 24 << 20)
    monkeypatch.setenv("SYMAR_TUNE", "exhaustive")
    g = symar.SymHeap.on_torch(8, 24 << 20)
    monkeypatch.delenv("SYMAR_TUNE")
    try:
        t0 = time.perf_counter()
        h.autotune(symar.BF16)
        quick = time.perf_counter() - t0
        t0 = time.perf_counter()
        g.autotune(symar.BF16)
        full = time.perf_counter() - t0
        assert quick < 5.0, (quick, full)
        for B in w["batch"]:
            count = w["count"] * B
            log2 = (count * 2 - 1).bit_length()
            algo = h.query_choice(count, symar.BF16)[0]
            mine = h.tuned_entry(symar.BF16, log2, algo)[2]
            best = min(g.tuned_entry(symar.BF16, log2, a)[2] for a in ALGOS[:-1])
            assert mine <= 1.08 * best, (B, algo, mine, best)
            # and it is the same algorithm, unless two are within that noise of each other
            theirs = g.query_choice(count, symar.BF16)[0]
            assert algo == theirs or g.tuned_entry(symar.BF16, log2, algo)[2] <= 1.08 * best, (B, algo, theirs)
    finally:
        torch.cuda.synchronize()
        h.destroy()
        g.destroy()


def test_c4_full_size_p8_fp32_256MiB():
    w = synth.WORKLOADS["c4"]
    P, count = w["P"], w["count"]
    M = count * 4
    x = synth.make_inputs(w["dist"], "f32", P, count, w["seed"])
    want = O.allreduce_timed_team(x, threads=0)[0][0]          # all rows of the oracle's output are equal
    h = symar.SymHeap.on_torch(P, 2 * M)
    try:
        for q in range(P):
            h.write_rank(q, 0, x[q])
        del x
        h.allreduce(0, M, count, symar.F32, symar.TWOSHOT)      # bench.py's call, default launch shape
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        assert h.last_kernel() == (4, 0)                         # the register kernel of the bandwidth regime ran
        want_bits = want.view(np.uint32)

        def check_all(what):
            for r in range(P):
                got = h.read_rank(r, M, count, np.float32).view(np.uint32)
                bad = np.flatnonzero(got != want_bits)
                assert bad.size == 0, f"{what}, rank {r}: {bad.size} mismatches, first at {bad[0]}"
                h.write_rank(r, M, np.zeros(1 << 20, dtype=np.uint8))      # stale results must not pass the next check

        check_all("default shape")
        # the bulk-copy kernel: 12 CTAs per rank, two stages of eight 8 KiB tiles
        h.set_launch(symar.TWOSHOT, 12, 256)
        h.set_variant(symar.TWOSHOT, (2 << 8) | (1 << 12))
        h.allreduce(0, M, count, symar.F32, symar.TWOSHOT)
        torch.cuda.synchronize()
        assert h.last_kernel()[1] > 0 and h.last_choice() == (symar.TWOSHOT, 12, 256)
        check_all("bulk-copy kernel 12 x 256")
        # the register kernel in another shape the tuner tends to pick for this size
        h.set_launch(symar.TWOSHOT, 15, 512)
        h.set_variant(symar.TWOSHOT, 4)
        h.allreduce(0, M, count, symar.F32, symar.TWOSHOT)
        torch.cuda.synchronize()
        assert h.last_kernel()[1] == 0 and h.last_choice() == (symar.TWOSHOT, 15, 512)
        check_all("register kernel 15 x 512")
        h.set_launch(symar.TWOSHOT, 0, 0)
        h.set_variant(symar.TWOSHOT, 0)
        # and exactly what bench.py times: the shape tuned for this size on this GPU (tuning overwrites
        # the user region, so the inputs go in again)
        x = synth.make_inputs(w["dist"], "f32", P, count, w["seed"])
        h.autotune_size(symar.F32, count)
        for q in range(P):
            h.write_rank(q, 0, x[q])
        del x
        h.allreduce(0, M, count, symar.F32, symar.TWOSHOT)
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        check_all(f"tuned shape {h.last_choice()} kernel {h.last_kernel()}")
    finally:
        h.destroy()


@pytest.mark.parametrize("P", [8, 4])
def test_c5_decode_trace_160_calls_in_one_graph(P):
    w = synth.WORKLOADS["c5"]
    calls, count = w["calls"], w["count"]
    nb = count * 2
    xs = [synth.make_inputs(w["dist"], "bf16", P, count, w["seed"], call=k) for k in range(calls)]
    wants = [O.allreduce(x)[0] for x in xs]
    h = symar.SymHeap.on_torch(P, 24 << 20)
    try:
        h.autotune(symar.BF16)                                   # as bench.py does before capturing
        for k in range(calls):
            for q in range(P):
                h.write_rank(q, k * nb, xs[k][q])
        out0 = 10 << 20
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=s):
            for k in range(calls):
                h.allreduce(k * nb, out0 + k * nb, count, symar.BF16, symar.AUTO, s.cuda_stream)
        for rep in range(3):
            for q in range(P):
                h.write_rank(q, out0, np.zeros(calls * nb, dtype=np.uint8))
            g.replay()
            torch.cuda.synchronize()
            assert h.status()[0] == symar.OK
            for q in range(P):
                got = h.read_rank(q, out0, calls * count, np.uint16).reshape(calls, count)
                for k in range(calls):
                    assert np.array_equal(got[k], wants[k]), (rep, q, k)
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_speed_of_light_probes_return_plausible_values():
    """The pieces of the latency bound (Sec. VI): every probe ends by itself and gives sub-10-us figures."""
    fence = symar.probe_fence(2000)
    assert 10.0 < fence < 10_000.0
    rt, sm = symar.probe_pingpong_pair(1, 2000)
    assert 50.0 < rt < 10_000.0 and sm[0] != sm[1]
    nsm = torch.cuda.get_device_properties(0).multi_processor_count
    rt2, sm2 = symar.probe_pingpong_blocks(nsm // 2, 3, nsm, 2000)
    assert 50.0 < rt2 < 10_000.0 and sm2[0] != sm2[1]
    with pytest.raises(symar.SymarError):
        symar.probe_pingpong_blocks(5, 5, nsm, 100)              # a block cannot play against itself
    with pytest.raises(symar.SymarError):
        symar.probe_pingpong_blocks(0, nsm, nsm, 100)            # partner outside the launch
    for ordered in (False, True):
        assert 50.0 < symar.probe_barrier(8, 500, ordered) < 20_000.0
    with pytest.raises(symar.SymarError):
        symar.probe_barrier(1, 10)
    s = torch.cuda.Stream()
    symar.probe_empty(4, 8, 128, s.cuda_stream)
    symar.probe_empty_pdl(4, 8, 128, s.cuda_stream)
    s.synchronize()


def test_environment_overrides_are_read_at_heap_creation(monkeypatch, capfd):
    monkeypatch.setenv("SYMAR_ALGO", "sentinel")
    monkeypatch.setenv("SYMAR_CTAS_PER_RANK", "3")
    monkeypatch.setenv("SYMAR_THREADS", "96")
    monkeypatch.setenv("SYMAR_PDL", "0")
    monkeypatch.setenv("SYMAR_DEBUG", "1")
    h = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        x = synth.make_inputs("normal", "bf16", 4, 3000, seed=5)
        for q in range(4):
            h.write_rank(q, 0, x[q])
        h.allreduce(0, 1 << 19, 3000, symar.BF16, symar.AUTO)
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        assert h.last_choice() == (symar.SENTINEL, 3, 96)
        got = np.stack([h.read_rank(q, 1 << 19, 3000, np.uint16) for q in range(4)])
        assert np.array_equal(got, O.allreduce(x))
        err = capfd.readouterr().err
        assert "symar: allreduce count=3000" in err and "pdl=0" in err and "block=96" in err
    finally:
        torch.cuda.synchronize()
        h.destroy()
    # and nothing is printed without SYMAR_DEBUG
    monkeypatch.delenv("SYMAR_DEBUG")
    h = symar.SymHeap.on_torch(2, 1 << 16)
    try:
        h.allreduce(0, 1 << 15, 16, symar.F32, symar.ONESHOT)
        torch.cuda.synchronize()
        assert capfd.readouterr().err == ""
    finally:
        h.destroy()


def test_in_kernel_span_hook_measures_and_keeps_results():
    h = symar.SymHeap.on_torch(8, 1 << 20)
    try:
        x = synth.make_inputs("normal", "bf16", 8, 8192, seed=2)
        for q in range(8):
            h.write_rank(q, 0, x[q])
        want = O.allreduce(x)
        for algo in (symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL,
                     symar.TWOSHOT_SENTINEL):
            spans = [h.debug_span(0, 1 << 19, 8192, symar.BF16, algo) for _ in range(5)]
            assert all(100.0 <= s <= 200_000.0 for s in spans), (algo, spans)     # 0.1 us ... 0.2 ms
            got = np.stack([h.read_rank(q, 1 << 19, 8192, np.uint16) for q in range(8)])
            assert np.array_equal(got, want), algo
        assert h.debug_span(0, 1 << 19, 8192, symar.BF16, symar.TWOSHOT_ATOMIC) > 0
        assert h.status()[0] == symar.OK
    finally:
        torch.cuda.synchronize()
        h.destroy()
