"""GPU parity: the CUDA AllReduce (through the C ABI) against the CPU oracle,
element by element and bit for bit, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import symar, synth

pytestmark = pytest.mark.gpu

ALGOS = [symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL]
NP_DT = {symar.F32: np.float32, symar.BF16: np.uint16}
DT = {"f32": symar.F32, "bf16": symar.BF16}
USER = 8 << 20          # user region per rank of the shared test heaps


@pytest.fixture(scope="module")
def heaps():
    hs = {P: symar.SymHeap.on_torch(P, USER) for P in (1, 2, 4, 8)}
    yield hs
    torch.cuda.synchronize()
    for h in hs.values():
        h.destroy()


def run(h, x, dtype, algo, in_off=0, out_off=None, stream=0, poison=True):
    """Upload x[P, count], run one allreduce, return out[P, count]."""
    P, count = x.shape
    nbytes = x.nbytes // P
    if out_off is None:
        out_off = (in_off + nbytes + 255) // 256 * 256
    if poison:
        for q in range(P):
            h.write_rank(q, out_off, np.full(nbytes + 64, 0xA5, dtype=np.uint8))
    for q in range(P):
        h.write_rank(q, in_off, x[q])
    h.allreduce(in_off, out_off, count, dtype, algo, stream)
    torch.cuda.synchronize()
    code = h.status()[0]
    assert code == symar.OK, f"device status {h.status()}"
    out = np.stack([h.read_rank(q, out_off, count, NP_DT[dtype]) for q in range(P)])
    if poison:   # nothing may be written past the end of the message
        for q in range(P):
            guard = h.read_rank(q, out_off + nbytes, 64, np.uint8)
            assert np.all(guard == 0xA5), f"rank {q}: wrote past the end of the output"
    return out


def assert_bits(got, want, what=""):
    if got.dtype == np.float32:
        got, want = got.view(np.uint32), want.view(np.uint32)
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{what}: {len(bad)} mismatches, first at [rank, i] = {bad[0]}: " \
                          f"got {got[tuple(bad[0])]:#x} want {want[tuple(bad[0])]:#x}"


# ---- tier 1: small shapes, every algorithm x dtype x P x ragged counts -------------

@pytest.mark.parametrize("count", [1, 3, 7, 8, 9, 31, 1023, 1024, 1025, 8191, 70001])
@pytest.mark.parametrize("P", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
@pytest.mark.parametrize("algo", ALGOS)
def test_small_shapes(heaps, algo, dtype, dist, P, count):
    x = synth.make_inputs(dist, dtype, P, count, seed=1000 + count)
    got = run(heaps[P], x, DT[dtype], algo)
    assert_bits(got, O.allreduce(x), f"algo={algo} {dtype} P={P} count={count}")


@pytest.mark.parametrize("algo", ALGOS)
def test_nonzero_offsets(heaps, algo):
    h = heaps[4]
    x = synth.make_inputs("normal", "bf16", 4, 5000, seed=77)
    got = run(h, x, symar.BF16, algo, in_off=4096 + 16, out_off=1 << 20)
    assert_bits(got, O.allreduce(x))
    # output placed BEFORE the input
    got = run(h, x, symar.BF16, algo, in_off=2 << 20, out_off=48)
    assert_bits(got, O.allreduce(x))


# ---- special values -----------------------------------------------------------------

@pytest.mark.parametrize("algo", ALGOS)
def test_special_values_f32(heaps, algo):
    sp = np.array([0.0, -0.0, 1e-45, -1e-45, 1.17549435e-38, np.inf, -np.inf, 3.4e38, -3.4e38, 1.0, 1e8, -1e8],
                  dtype=np.float32)
    rng = np.random.default_rng(3)
    x = sp[rng.integers(0, len(sp), size=(4, 4096))]
    got = run(heaps[4], x, symar.F32, algo)
    want = O.allreduce(x)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert_bits(np.where(nan, np.float32(0), got), np.where(nan, np.float32(0), want))


@pytest.mark.parametrize("algo", ALGOS)
def test_special_values_bf16(heaps, algo):
    sp = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x0080, 0x7F80, 0xFF80, 0x7F7F, 0xFF7F, 0x3F80, 0x3B80,
                   0x4380, 0x7FC0], dtype=np.uint16)
    rng = np.random.default_rng(4)
    x = sp[rng.integers(0, len(sp), size=(8, 4096))]
    got = run(heaps[8], x, symar.BF16, algo)
    want = O.allreduce(x)
    is_nan = lambda h: ((h & 0x7F80) == 0x7F80) & ((h & 0x007F) != 0)
    assert np.array_equal(is_nan(got), is_nan(want))
    keep = ~is_nan(want)
    assert_bits(np.where(keep, got, 0), np.where(keep, want, 0))


def test_hand_case_order_pin_on_gpu(heaps):
    # rank order 0..3: (1 + 1e8) - 1e8 + 0 = 0 in binary32; a reordered sum gives 1
    x = np.array([[1.0] * 8, [1e8] * 8, [-1e8] * 8, [0.0] * 8], dtype=np.float32)
    for algo in ALGOS:
        got = run(heaps[4], x, symar.F32, algo)
        assert np.all(got == 0.0)
    got = run(heaps[4], x[::-1].copy(), symar.F32, symar.LL)
    assert np.all(got == 1.0)


# ---- launch shapes, multi-iteration LL ----------------------------------------------

@pytest.mark.parametrize("ctas,threads", [(1, 32), (1, 512), (3, 64), (7, 96), (16, 256), (64, 128)])
@pytest.mark.parametrize("algo", ALGOS)
def test_forced_launch_shapes(heaps, algo, ctas, threads):
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 40009, seed=ctas * 1000 + threads)
    h.set_launch(algo, ctas, threads)
    try:
        got = run(h, x, symar.BF16, algo)
        a, c, t = h.last_choice()
        if algo in (symar.LL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL):
            # register-heavy kernels: at most 256 threads, and the library clamps the grid to
            # what is co-resident (CTAs of different ranks wait for one another)
            assert a == algo and t == min(threads, 256) and 1 <= c <= ctas
        else:
            assert (a, c, t) == (algo, ctas, threads)
    finally:
        h.set_launch(algo, 0, 0)
    assert_bits(got, O.allreduce(x))


@pytest.mark.parametrize("algo", [symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL])
def test_push_many_iterations_alternate_subbuffers(heaps, algo):
    # one CTA per rank, 1024 vectors per iteration: 300000 fp32 -> 75000 vectors -> 74 iterations
    h = heaps[4]
    x = synth.make_inputs("uniform", "f32", 4, 300000, seed=5)
    h.set_launch(algo, 1, 256)
    try:
        got = run(h, x, symar.F32, algo)
        got2 = run(h, x[::-1].copy(), symar.F32, algo)      # straight again on the same scratch
    finally:
        h.set_launch(algo, 0, 0)
    assert_bits(got, O.allreduce(x))
    assert_bits(got2, O.allreduce(x[::-1].copy()))


@pytest.mark.parametrize("algo", [symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL])
@pytest.mark.parametrize("limit", [16, 4096, 100000])
def test_small_scratch_buffers_take_more_iterations(heaps, algo, limit):
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 90001, seed=limit)
    h.set_scratch_limit(limit)
    try:
        got = run(h, x, symar.BF16, algo)
    finally:
        h.set_scratch_limit(0)
    assert_bits(got, O.allreduce(x), f"algo {algo} scratch {limit}")


def test_sentinel_mode_accepts_payload_equal_to_the_sentinel(heaps):
    # words of all ones (a negative NaN; in bf16 two of them) are the scratch's
    # sentinel; such payload is sent with one bit changed -- still NaN -- so the
    # receiver is never left waiting and NaN-ness of the result is kept
    h = heaps[8]
    rng = np.random.default_rng(8)
    x = synth.make_inputs("uniform", "f32", 8, 4096, seed=3)
    xw = x.view(np.uint32)
    xw[rng.integers(0, 8, 300), rng.integers(0, 4096, 300)] = 0xFFFFFFFF
    want = O.allreduce(x)
    for algo in (symar.SENTINEL, symar.TWOSHOT_SENTINEL):
        got = run(h, x, symar.F32, algo)
        assert np.array_equal(np.isnan(got), np.isnan(want)) and np.isnan(want).sum() >= 250
        keep = ~np.isnan(want)
        assert_bits(np.where(keep, got, np.float32(0)), np.where(keep, want, np.float32(0)))
        for q in range(1, 8):                 # every rank holds the same bits, NaN payloads included
            assert np.array_equal(got[q].view(np.uint32), got[0].view(np.uint32))
    xb = synth.make_inputs("normal", "bf16", 8, 4096, seed=4)
    xb.view(np.uint32)[rng.integers(0, 8, 200), rng.integers(0, 2048, 200)] = 0xFFFFFFFF
    wantb = O.allreduce(xb)
    gotb = run(h, xb, symar.BF16, symar.SENTINEL)
    is_nan = lambda v: ((v & 0x7F80) == 0x7F80) & ((v & 0x007F) != 0)
    assert np.array_equal(is_nan(gotb), is_nan(wantb))
    assert_bits(np.where(is_nan(wantb), 0, gotb), np.where(is_nan(wantb), 0, wantb))
    # and the scratch is whole again afterwards
    y = synth.make_inputs("normal", "bf16", 8, 4096, seed=5)
    assert_bits(run(h, y, symar.BF16, symar.SENTINEL), O.allreduce(y))


FORCE_PLAIN = 1 << 31
CLUSTER = symar.VARIANT_CLUSTER


@pytest.mark.parametrize("count", [1, 2, 3, 5, 8, 9, 63, 64, 1023, 4099, 40001])
@pytest.mark.parametrize("P,dtype,dist", [(8, "bf16", "normal"), (4, "f32", "uniform"), (2, "bf16", "normal"),
                                          (1, "f32", "uniform")])
@pytest.mark.parametrize("algo,variant", [(symar.ONESHOT, FORCE_PLAIN), (symar.ONESHOT, 0x100),
                                          (symar.ONESHOT, 0x200),
                                          # release on the ready signal (comparison variant)
                                          (symar.ONESHOT, 0x8100), (symar.ONESHOT, 0x8000),
                                          # LL: single-iteration kernel where it fits (16 / 8 payload bytes per
                                          # thread, first poll held back), and the general kernel (bit 9)
                                          (symar.LL, FORCE_PLAIN), (symar.LL, 0x100), (symar.LL, 0x3100),
                                          (symar.LL, 0xC000), (symar.LL, 0x200), (symar.LL, 0x300),
                                          (symar.SENTINEL, FORCE_PLAIN), (symar.TWOSHOT_LL, FORCE_PLAIN),
                                          (symar.TWOSHOT_SENTINEL, FORCE_PLAIN),
                                          # two-shot: 16 or 8 bytes per thread and trip
                                          (symar.TWOSHOT, FORCE_PLAIN), (symar.TWOSHOT, 0x40),
                                          # the ranks of a slot launched as one thread-block cluster
                                          (symar.ONESHOT, CLUSTER | 0x100), (symar.ONESHOT, CLUSTER),
                                          (symar.TWOSHOT, CLUSTER), (symar.TWOSHOT, CLUSTER | 0x40),
                                          (symar.LL, CLUSTER | 0x100), (symar.LL, CLUSTER | 0x2100),
                                          (symar.LL, CLUSTER | 0x200), (symar.SENTINEL, CLUSTER),
                                          (symar.TWOSHOT_LL, CLUSTER), (symar.TWOSHOT_SENTINEL, CLUSTER)])
def test_unit_width_variants(heaps, algo, variant, P, dtype, dist, count):
    # every implementation variant of a kernel gives the same bits, whatever the ragged tail
    h = heaps[P]
    x = synth.make_inputs(dist, dtype, P, count, seed=31 * count + P)
    h.set_variant(algo, variant)
    try:
        got = run(h, x, DT[dtype], algo)
        # (a cluster needs two ranks at least, and all clusters of a launch must be resident together:
        # otherwise the same shape is launched plainly; the small launches here always fit)
        asked = variant & 0x7FFFFFFF
        if P == 1:
            asked &= ~CLUSTER
        assert h.last_kernel()[0] in ((asked,) if count < 5000 else (asked, asked & ~CLUSTER))
    finally:
        h.set_variant(algo, 0)
    assert_bits(got, O.allreduce(x), f"algo={algo} variant={variant:#x} P={P} {dtype} count={count}")


def test_cluster_launch_falls_back_when_the_clusters_do_not_fit(heaps):
    # 160 CTAs of 512 threads per rank cannot all be resident as clusters of eight (nor as plain CTAs): the
    # library shrinks the grid to what fits and launches it plainly if the clusters still do not fit; a
    # shape that fits keeps its clusters.  Same bits either way.
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 300001, seed=123)
    want = O.allreduce(x)
    try:
        for algo in (symar.ONESHOT, symar.TWOSHOT):
            h.set_variant(algo, CLUSTER)
            h.set_launch(algo, 160, 512)
            assert_bits(run(h, x, symar.BF16, algo), want, f"algo {algo}, 160 x 512")
            big = h.last_kernel()[0] & CLUSTER
            h.set_launch(algo, 8, 128)
            assert_bits(run(h, x, symar.BF16, algo), want, f"algo {algo}, 8 x 128")
            assert h.last_kernel()[0] & CLUSTER and h.last_choice()[1:] == (8, 128)
            assert big in (0, CLUSTER)
    finally:
        for algo in (symar.ONESHOT, symar.TWOSHOT):
            h.set_variant(algo, 0)
            h.set_launch(algo, 0, 0)


def test_ll_narrow_many_iterations_and_mixed_widths(heaps):
    # narrow and wide LL calls alternate on the same scratch; one CTA forces many iterations
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 100003, seed=77)
    want = O.allreduce(x)
    try:
        for variant, ctas, threads in ((0x100, 1, 128), (FORCE_PLAIN, 2, 64), (0x100, 3, 512), (0x100, 64, 32)):
            h.set_variant(symar.LL, variant)
            h.set_launch(symar.LL, ctas, threads)
            assert_bits(run(h, x, symar.BF16, symar.LL, poison=False), want, f"variant {variant:#x}")
    finally:
        h.set_variant(symar.LL, 0)
        h.set_launch(symar.LL, 0, 0)


# ---- bandwidth regime: block-cyclic ownership, 32-byte accesses, bulk-copy pipeline ----

@pytest.fixture(scope="module")
def big_heaps():
    hs = {P: symar.SymHeap.on_torch(P, 40 << 20) for P in (2, 4, 8)}
    yield hs
    torch.cuda.synchronize()
    for h in hs.values():
        h.destroy()


def bulk_var(stages, tile_log2):
    return (stages << 8) | (tile_log2 << 12)


@pytest.mark.parametrize("P,dtype,count", [
    (8, "f32", 1 << 20), (8, "f32", (1 << 20) + 1), (8, "f32", (1 << 20) + 2051), (8, "bf16", (1 << 21) + 5),
    (8, "bf16", 3 * (1 << 20) + 4099), (4, "f32", (1 << 20) + 7), (2, "bf16", (1 << 21) + 8193),
    (8, "f32", 4 * (1 << 20) + 3),
])
@pytest.mark.parametrize("variant,ctas,threads", [
    (0, 0, 0),                       # defaults: register kernel, 512 threads per SM in all
    (bulk_var(2, 0), 12, 256),       # bulk kernel, 64 KiB stage among eight ranks
    (bulk_var(3, 0), 37, 256),       # 4 KiB tiles, three stages, two CTAs per SM
    (bulk_var(2, 1), 7, 128),        # 8 KiB tiles, odd CTA count
    (bulk_var(4, 0), 13, 512),
    (bulk_var(2, 3), 3, 64),         # tile larger than shared memory allows: library shrinks it
    (4, 37, 256),                    # register kernel: block-cyclic + 32-byte accesses
    (4 | 2, 18, 512),                # register kernel: block-cyclic, 16-byte accesses
    (4 | 1, 5, 96),                  # register kernel: one contiguous chunk per rank
])
def test_bandwidth_regime_paths(big_heaps, P, dtype, count, variant, ctas, threads):
    h = big_heaps[P]
    dist = "uniform" if dtype == "f32" else "normal"
    x = synth.make_inputs(dist, dtype, P, count, seed=count + P)
    out_off = 20 << 20
    h.set_variant(symar.TWOSHOT, variant)
    h.set_launch(symar.TWOSHOT, ctas, threads)
    try:
        got = run(h, x, DT[dtype], symar.TWOSHOT, in_off=0, out_off=out_off)
        var, smem = h.last_kernel()
        if variant == 0:
            assert smem == 0 and (var & 4), "the default of the bandwidth regime is the register kernel"
        elif not (variant & 4):
            assert smem > 0, "the bulk-copy kernel should have been used"
        else:
            assert smem == 0
    finally:
        h.set_variant(symar.TWOSHOT, 0)
        h.set_launch(symar.TWOSHOT, 0, 0)
    assert_bits(got, O.allreduce(x), f"P={P} {dtype} count={count} variant={variant:#x}")


def test_bandwidth_regime_unaligned_buffers(big_heaps):
    # 16-byte (not 32-byte) aligned input and output: bulk copies still legal, the
    # register kernel must fall back to 16-byte accesses
    h = big_heaps[8]
    count = (1 << 20) + 37
    x = synth.make_inputs("uniform", "f32", 8, count, seed=4242)
    for variant in (bulk_var(2, 1), 4):
        h.set_variant(symar.TWOSHOT, variant)
        try:
            got = run(h, x, symar.F32, symar.TWOSHOT, in_off=16, out_off=(20 << 20) + 48)
        finally:
            h.set_variant(symar.TWOSHOT, 0)
        assert_bits(got, O.allreduce(x), f"variant {variant}")


# sizes at which the built-in algorithm, the unit width or the rule for the launch shape changes
BOUNDARY_BYTES = [256, 272, 2048, 2064, 8192, 8208, 65536, 65552, 262144, 262160, 524288, 524304, (1 << 20) - 16,
                  1 << 20, (1 << 20) + 48, (2 << 20) + 4112, (4 << 20) - 16, 4 << 20, (4 << 20) + 16]


@pytest.mark.parametrize("nbytes", BOUNDARY_BYTES)
@pytest.mark.parametrize("P", [2, 4, 8])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_builtin_choices_at_their_boundaries(big_heaps, P, dtype, nbytes):
    """No tuning, no forced shape: what a first call gets, on both sides of every threshold."""
    h = big_heaps[P]
    es = 4 if dtype == "f32" else 2
    for count in (nbytes // es, nbytes // es - 1):
        x = synth.make_inputs("uniform" if dtype == "f32" else "normal", dtype, P, count, seed=nbytes + P)
        want = O.allreduce(x)
        for algo in (symar.AUTO, symar.ONESHOT, symar.TWOSHOT):
            got = run(h, x, DT[dtype], algo, in_off=0, out_off=20 << 20)
            assert_bits(got, want, f"P={P} {dtype} count={count} algo={algo} launched {h.last_choice()}")


# ---- determinism, algorithm equality, interleaving stress ---------------------------

def test_algorithms_agree_and_repeat(heaps):
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 8192, seed=synth.seed_for_config(2))
    want = O.allreduce(x)
    for rep in range(40):
        for algo in ALGOS:
            assert_bits(run(h, x, symar.BF16, algo, poison=(rep == 0)), want, f"rep {rep} algo {algo}")


@pytest.mark.parametrize("algo", ALGOS)
def test_seeded_start_delays_do_not_change_results(heaps, algo):
    h = heaps[8]
    x = synth.make_inputs("uniform", "f32", 8, 20000, seed=31)
    want = O.allreduce(x)
    try:
        for seed in range(12):
            h.debug_inject(-1, seed + 1, 20000)          # every CTA starts up to 20 us late
            assert_bits(run(h, x, symar.F32, algo, poison=False), want, f"delay seed {seed}")
    finally:
        h.debug_inject(-1, 0, 0)


def test_mixed_algorithms_and_shapes_share_flags_safely(heaps):
    # successive calls with different algorithms, sizes and grids reuse the same
    # flag words and scratch; per-slot counters must keep every flag value fresh
    h = heaps[8]
    rng = np.random.default_rng(12)
    for i in range(60):
        algo = ALGOS[int(rng.integers(0, len(ALGOS)))]
        count = int(rng.integers(1, 30000))
        dtype = ("f32", "bf16")[int(rng.integers(0, 2))]
        h.set_launch(algo, int(rng.integers(1, 40)), int(rng.choice([32, 64, 128, 256, 512])))
        x = synth.make_inputs("normal", dtype, 8, count, seed=500 + i)
        try:
            got = run(h, x, DT[dtype], algo, poison=False)
        finally:
            h.set_launch(algo, 0, 0)
        assert_bits(got, O.allreduce(x), f"step {i} algo {algo} count {count}")


# ---- CUDA graph capture and replay ----------------------------------------------------

def test_graph_capture_replays(heaps):
    h = heaps[8]
    count, calls = 8192 * 4, 6
    nbytes = count * 2
    xs = [synth.make_inputs("normal", "bf16", 8, count, seed=synth.seed_for_config(5), call=k)
          for k in range(calls)]
    for k, x in enumerate(xs):
        for q in range(8):
            h.write_rank(q, k * nbytes, x[q])
    out0 = 4 << 20
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g, stream=s):
        for k in range(calls):
            algo = ALGOS[k % len(ALGOS)]
            h.allreduce(k * nbytes, out0 + k * nbytes, count, symar.BF16, algo, s.cuda_stream)
    for rep in range(4):
        for q in range(8):
            h.write_rank(q, out0, np.zeros(calls * nbytes, dtype=np.uint8))
        g.replay()
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        for k, x in enumerate(xs):
            want = O.allreduce(x)
            got = np.stack([h.read_rank(q, out0 + k * nbytes, count, np.uint16) for q in range(8)])
            assert_bits(got, want, f"replay {rep} call {k}")


@pytest.mark.parametrize("pdl", [True, False])
def test_programmatic_dependent_launch_keeps_results_and_order(heaps, pdl):
    # back-to-back calls whose input is the previous call's output: with the
    # launch attribute on, each kernel may become resident early but must not
    # touch the heap before its predecessor has finished
    h = heaps[8]
    count = 8192
    nb = count * 2
    x = synth.make_inputs("normal", "bf16", 8, count, seed=606)
    for q in range(8):
        h.write_rank(q, 0, x[q])
    h.set_pdl(pdl)                              # on is the default; off must give the same
    try:
        s = torch.cuda.Stream()
        chain = [ALGOS[k % len(ALGOS)] for k in range(9)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for k, algo in enumerate(chain):
                h.allreduce(k * nb, (k + 1) * nb, count, symar.BF16, algo, s.cuda_stream)
        for rep in range(3):
            g.replay()
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        want = x
        for k in range(len(chain)):
            want = O.allreduce(want)            # every rank's next input is the previous result
            got = np.stack([h.read_rank(q, (k + 1) * nb, count, np.uint16) for q in range(8)])
            assert_bits(got, want, f"link {k}")
        # stream-launched as well
        for algo in ALGOS:
            got = run(h, x, symar.BF16, algo, in_off=0, out_off=1 << 20, poison=False)
            assert_bits(got, O.allreduce(x))
    finally:
        h.set_pdl(True)


# ---- AUTO, autotune -----------------------------------------------------------------------

def test_auto_default_and_after_autotune():
    h = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        x = synth.make_inputs("int_pm8", "f32", 4, 1024, seed=synth.seed_for_config(1))
        got = run(h, x, symar.F32, symar.AUTO)
        assert_bits(got, O.allreduce(x))
        assert h.last_choice()[0] in ALGOS
        h.autotune(symar.F32)
        for count in (4, 1024, 70000, 131072):
            x = synth.make_inputs("uniform", "f32", 4, count, seed=count)
            got = run(h, x, symar.F32, symar.AUTO, poison=False)
            assert_bits(got, O.allreduce(x))
            a, c, t = h.last_choice()
            assert (a, c, t) == h.query_choice(count, symar.F32)
        row = h.tuned_entry(symar.F32, 14, symar.LL)
        assert row is not None and row[0] >= 1 and row[2] > 0
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_autotune_of_one_size_fills_only_its_bucket(tmp_path):
    h = symar.SymHeap.on_torch(4, 1 << 20)
    g = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        count = 3 * 4096 + 5                                     # 49172 B of f32: bucket 16 (the next power of two)
        before = h.query_choice(1024, symar.F32)
        h.autotune_size(symar.F32, count)
        assert h.tuned_entry(symar.F32, 16, symar.ONESHOT) is not None
        assert h.tuned_entry(symar.F32, 15, symar.ONESHOT) is None      # other buckets untouched
        assert h.query_choice(1024, symar.F32) == before                # and still on the defaults
        a, c, t = h.query_choice(count, symar.F32)
        best = min(ALGOS, key=lambda algo: h.tuned_entry(symar.F32, 16, algo)[2])
        assert a == best and (c, t) == h.tuned_entry(symar.F32, 16, a)[:2]
        x = synth.make_inputs("normal", "f32", 4, count, seed=3)
        assert_bits(run(h, x, symar.F32, symar.AUTO), O.allreduce(x))
        assert h.last_choice() == (a, c, t)
        # survives a file round trip without a grid table beside it
        path = tmp_path / "one.txt"
        h.table_save(path)
        g.table_load(path)
        assert g.query_choice(count, symar.F32) == (a, c, t)
        assert g.tuned_entry(symar.F32, 15, symar.ONESHOT) is None
        # a later full tuning keeps nothing stale inside its grid and stays bit-exact
        h.autotune(symar.F32)
        assert h.tuned_entry(symar.F32, 15, symar.ONESHOT) is not None
        assert_bits(run(h, x, symar.F32, symar.AUTO, poison=False), O.allreduce(x))
        with pytest.raises(symar.SymarError):
            h.autotune_size(symar.F32, (1 << 20) // 4)          # input and output would not fit
        with pytest.raises(symar.SymarError):
            h.autotune_size(symar.F32, 0)
    finally:
        torch.cuda.synchronize()
        h.destroy()
        g.destroy()


def test_autotune_for_a_stream_of_calls_with_their_own_buffers():
    # the tuner's streaming mode: every timed call on its own input / output pair, as in a decode step
    h = symar.SymHeap.on_torch(4, 4 << 20)
    try:
        count = 8192                                             # 16 KiB of bf16: bucket 14
        before = h.query_choice(300, symar.BF16)
        h.autotune_stream(symar.BF16, count, 24)                 # 24 pairs of 16 KiB = 768 KiB of the 4 MiB region
        assert h.tuned_entry(symar.BF16, 14, symar.ONESHOT) is not None
        assert h.tuned_entry(symar.BF16, 13, symar.ONESHOT) is None
        assert h.query_choice(300, symar.BF16) == before
        a, c, t = h.query_choice(count, symar.BF16)
        assert a in ALGOS and (c, t) == h.tuned_entry(symar.BF16, 14, a)[:2]
        x = synth.make_inputs("normal", "bf16", 4, count, seed=21)
        assert_bits(run(h, x, symar.BF16, symar.AUTO), O.allreduce(x))
        assert h.last_choice() == (a, c, t)
        with pytest.raises(symar.SymarError):
            h.autotune_stream(symar.BF16, count, 200)            # 200 pairs do not fit
        with pytest.raises(symar.SymarError):
            h.autotune_stream(symar.BF16, count, 1)
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_tuned_table_round_trips_through_a_file(tmp_path):
    a = symar.SymHeap.on_torch(4, 1 << 18)
    b = symar.SymHeap.on_torch(4, 1 << 18)
    c = symar.SymHeap.on_torch(2, 1 << 18)
    try:
        a.autotune(symar.BF16)
        path = tmp_path / "table.txt"
        a.table_save(path)
        b.table_load(path)
        for count in (8, 512, 8192, 50000):
            assert a.query_choice(count, symar.BF16) == b.query_choice(count, symar.BF16)
        for log2 in range(4, 17):
            for algo in ALGOS:
                assert a.tuned_entry(symar.BF16, log2, algo)[:2] == b.tuned_entry(symar.BF16, log2, algo)[:2]
        with pytest.raises(symar.SymarError):
            c.table_load(path)                       # written for another rank count
        bad = tmp_path / "bad.txt"
        bad.write_text("symar-table 1 P 4\ndtype 1 buckets 4 6\ncfg 5 2 9999 64 0 1.0\n")
        with pytest.raises(symar.SymarError):
            b.table_load(bad)
        x = synth.make_inputs("normal", "bf16", 4, 8192, seed=1)
        assert_bits(run(b, x, symar.BF16, symar.AUTO, in_off=0, out_off=1 << 17), O.allreduce(x))
    finally:
        torch.cuda.synchronize()
        for h in (a, b, c):
            h.destroy()


# ---- errors --------------------------------------------------------------------------------

def test_argument_errors(heaps):
    h = heaps[4]
    rc = h.allreduce_rc
    assert rc(0, 4096, 0, symar.F32, symar.LL) == symar.OK                       # count 0: no-op
    assert rc(8, 4096, 16, symar.F32, symar.LL) == symar.ERR_INVAL               # misaligned in
    assert rc(0, 4100, 16, symar.F32, symar.LL) == symar.ERR_INVAL               # misaligned out
    assert rc(0, 32, 16, symar.F32, symar.LL) == symar.ERR_INVAL                 # overlap
    assert rc(0, 0, 16, symar.F32, symar.LL) == symar.ERR_INVAL                  # in place
    assert rc(0, USER - 16, 16, symar.F32, symar.LL) == symar.ERR_INVAL          # runs off the region
    assert rc(USER, 0, 4, symar.F32, symar.LL) == symar.ERR_INVAL
    assert rc(0, 4096, 16, 7, symar.LL) == symar.ERR_INVAL                       # dtype
    assert rc(0, 4096, 16, symar.F32, 9) == symar.ERR_INVAL                      # algo
    assert rc(0, 4096, 1 << 62, symar.F32, symar.LL) == symar.ERR_INVAL          # size overflow
    assert h.status()[0] == symar.OK
    with pytest.raises(symar.SymarError):
        h.rank_ptr(4, 0)
    with pytest.raises(symar.SymarError):
        symar.SymHeap(3, 4096)


@pytest.mark.parametrize("algo", ALGOS)
def test_bounded_wait_reports_timeout_and_heap_recovers(algo):
    # Rank 2 stays silent (host-requested test hook): its peers' waits run out
    # after the 2 ms limit, the kernel returns, the status word names the peer.
    h = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        x = synth.make_inputs("normal", "bf16", 4, 4096, seed=8)
        for q in range(4):
            h.write_rank(q, 0, x[q])
        h.set_spin_limit_us(2000)
        h.debug_inject(2, 0, 0)
        h.allreduce(0, 65536, 4096, symar.BF16, algo)
        torch.cuda.synchronize()
        code, rank, peer, cta = h.status()
        assert code == symar.ERR_TIMEOUT
        assert peer == 2 and rank != 2
        # recovery: clear the hook, reset flags/scratch/status, run again
        h.debug_inject(-1, 0, 0)
        h.reset()
        got = run(h, x, symar.BF16, algo)
        assert_bits(got, O.allreduce(x))
    finally:
        torch.cuda.synchronize()
        h.destroy()


@pytest.mark.parametrize("algo", [symar.ONESHOT, symar.LL, symar.TWOSHOT])
def test_default_wait_bound_is_a_fraction_of_a_second(algo):
    # With the library's default bound, a wait that can never end gives up well within a second
    # (a GPU that other work shares must not be held for long) and says so in the status word.
    import time
    h = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        x = synth.make_inputs("normal", "bf16", 4, 4096, seed=9)
        for q in range(4):
            h.write_rank(q, 0, x[q])
        h.debug_inject(1, 0, 0)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        h.allreduce(0, 65536, 4096, symar.BF16, algo)
        torch.cuda.synchronize()
        took = time.perf_counter() - t0
        assert h.status()[0] == symar.ERR_TIMEOUT
        assert 0.05 < took < 0.9, took
    finally:
        torch.cuda.synchronize()
        h.destroy()


@pytest.mark.parametrize("P", [2, 4, 8])
def test_placement_on_the_two_l2_halves_changes_no_bits(P):
    # Flags and counters are kept twice, one copy per half of the chip's L2; a reader takes the copy of its own
    # half when the heap could measure where things sit, copy 0 otherwise or when told so.  Calls with
    # placement on and off alternate on one heap (every call updates both copies): same bits as the oracle.
    h = symar.SymHeap.on_torch(P, 2 << 20)
    try:
        measured, sms_on_second_half, home = h.placement()
        if measured:                        # a B200: two halves, each with a good part of the SMs
            n = torch.cuda.get_device_properties(0).multi_processor_count
            assert n // 4 <= sms_on_second_half <= 3 * n // 4
        for i, (algo, count) in enumerate([(symar.ONESHOT, 8192), (symar.TWOSHOT, 8192), (symar.LL, 8192),
                                           (symar.ONESHOT, 77), (symar.TWOSHOT, 70001), (symar.LL, 1023),
                                           (symar.SENTINEL, 4099), (symar.TWOSHOT_LL, 4099), (symar.ONESHOT, 70001),
                                           (symar.TWOSHOT, 300000), (symar.ONESHOT, 8192), (symar.LL, 8192)]):
            h.set_placement(i % 2 == 0)
            x = synth.make_inputs("normal", "bf16", P, count, seed=500 + i)
            assert_bits(run(h, x, symar.BF16, algo), O.allreduce(x), f"placement {'on' if i % 2 == 0 else 'off'} {algo} {count}")
        # the sibling collectives share the flags and counters
        h.set_placement(True)
        x = synth.make_inputs("normal", "bf16", P, 4096 * P, seed=9)
        for q in range(P):
            h.write_rank(q, 0, x[q])
        assert h.reduce_scatter(0, 1 << 20, 4096, symar.BF16) == 0
        torch.cuda.synchronize()
        got = np.stack([h.read_rank(q, 1 << 20, 4096, np.uint16) for q in range(P)])
        assert np.array_equal(got, O.reduce_scatter(x)) and h.status()[0] == symar.OK
    finally:
        h.set_placement(True)
        torch.cuda.synchronize()
        h.destroy()


def test_placement_can_be_switched_off_in_the_environment(monkeypatch):
    monkeypatch.setenv("SYMAR_PLACE", "0")
    h = symar.SymHeap.on_torch(4, 1 << 18)
    try:
        assert h.placement() == (False, 0, 0)
        x = synth.make_inputs("normal", "bf16", 4, 8192, seed=3)
        assert_bits(run(h, x, symar.BF16, symar.ONESHOT, out_off=1 << 17), O.allreduce(x))
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_host_buffer_entry_point(heaps):
    h = heaps[8]
    count = 50000
    x = synth.make_inputs("uniform", "f32", 8, count, seed=91)
    hin = torch.from_numpy(x).pin_memory()
    hout = torch.empty_like(hin).pin_memory()
    h.allreduce_host(hin.data_ptr(), hout.data_ptr(), 0, 1 << 20, count, symar.F32, symar.AUTO)
    torch.cuda.synchronize()
    assert_bits(hout.numpy(), O.allreduce(x))


@pytest.mark.parametrize("dtype,count", [
    ("f32", 20 * (1 << 20) + 12345),      # 80 MiB per rank: 16 MiB chunks, the last one ragged
    ("f32", 25 * (1 << 20) + 12345),      # 100 MiB: seven chunks, 4 bytes past a 16-byte boundary
    ("bf16", 52 * (1 << 20) + 7),         # 104 MiB: an odd count of 2-byte elements
])
def test_host_buffer_entry_point_pipelines_large_messages(dtype, count):
    # cut into chunks that overlap transfers and kernels
    P = 2
    es = 4 if dtype == "f32" else 2
    M = count * es
    out_off = (M + 4095) // 4096 * 4096
    h = symar.SymHeap.on_torch(P, out_off + M)
    try:
        x = synth.make_inputs("uniform" if dtype == "f32" else "normal", dtype, P, count, seed=17)
        want = O.allreduce(x)
        hin = torch.from_numpy(x).pin_memory()
        hout = torch.empty_like(hin).pin_memory()
        s = torch.cuda.Stream()
        for rep in range(2):                                     # twice: the second call reuses the pipeline's events
            hout.zero_()
            h.allreduce_host(hin.data_ptr(), hout.data_ptr(), 0, out_off, count, DT[dtype], symar.AUTO, s.cuda_stream)
            s.synchronize()
            assert h.status()[0] == symar.OK
            assert_bits(hout.numpy(), want, f"rep {rep}")
        # the device copy of the result is complete as well
        got = np.stack([h.read_rank(q, out_off, count, NP_DT[DT[dtype]]) for q in range(P)])
        assert_bits(got, want)
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_capture_with_foreign_kernels_copies_and_the_host_pipeline():
    # every launch carries the programmatic-dependent-launch attribute by default: it must capture
    # behind kernels of other libraries and behind copy nodes, and the chunked host path must
    # fork and join its copy streams inside the capture
    P, count = 2, 9 * (1 << 20) + 77                             # 36 MiB per rank: three chunks
    M = count * 4
    out_off = (M + 4095) // 4096 * 4096
    h = symar.SymHeap.on_torch(P, out_off + M)
    try:
        x = synth.make_inputs("uniform", "f32", P, count, seed=23)
        small = np.ascontiguousarray(x[:, :6000])
        hin = torch.from_numpy(x).pin_memory()
        hout = torch.empty_like(hin).pin_memory()
        other = torch.zeros(1 << 16, device="cuda")
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            cs = torch.cuda.current_stream().cuda_stream
            other.fill_(1.0)                                     # a kernel of another library
            h.allreduce_host(hin.data_ptr(), hout.data_ptr(), 0, out_off, count, symar.F32, symar.AUTO, cs)
            other.add_(1.0)
            h.allreduce(0, out_off, 6000, symar.F32, symar.ONESHOT, cs)     # first 6000 elements again
        for _ in range(3):
            hout.zero_()
            g.replay()
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK and float(other[0]) == 2.0
        assert_bits(hout.numpy(), O.allreduce(x))
        got = np.stack([h.read_rank(q, out_off, 6000, np.float32) for q in range(P)])
        assert_bits(got, O.allreduce(small))
    finally:
        torch.cuda.synchronize()
        h.destroy()


def test_library_owned_heap():
    h = symar.SymHeap(2, 1 << 16)
    try:
        info = h.info()
        assert info.P == 2 and info.total_bytes == symar.required_bytes(2, 1 << 16)
        assert h.rank_ptr(1, 0) - h.rank_ptr(0, 0) == info.stride
    finally:
        h.destroy()


def test_prior_art_two_barrier_oneshot_gives_the_same_bits(heaps):
    # variant bit 14: the barrier-based form the method replaces, kept for comparison in the bench
    h = heaps[8]
    x = synth.make_inputs("normal", "bf16", 8, 8192, seed=14)
    try:
        for var in (0x4000, 0x4100, 0x4200):
            h.set_variant(symar.ONESHOT, var)
            for _ in range(3):
                assert_bits(run(h, x, symar.BF16, symar.ONESHOT, poison=False), O.allreduce(x), hex(var))
        h.set_variant(symar.ONESHOT, 0)
        assert_bits(run(h, x, symar.BF16, symar.TWOSHOT), O.allreduce(x))      # shares the done flags
    finally:
        h.set_variant(symar.ONESHOT, 0)


def test_symar_cluster_env_keeps_every_launch_plain(monkeypatch):
    # SYMAR_CLUSTER=0 (read when a heap is created): no launch carries the cluster attribute, whatever the
    # built-in rule or a forced variant says; results are the same bits
    monkeypatch.setenv("SYMAR_CLUSTER", "0")
    h = symar.SymHeap.on_torch(4, 1 << 20)
    monkeypatch.delenv("SYMAR_CLUSTER")
    g = symar.SymHeap.on_torch(4, 1 << 20)
    try:
        x = synth.make_inputs("normal", "bf16", 4, 3001, seed=66)
        want = O.allreduce(x)
        for algo in (symar.LL, symar.ONESHOT):
            assert_bits(run(h, x, symar.BF16, algo), want)
            assert not h.last_kernel()[0] & CLUSTER
            h.set_variant(algo, CLUSTER | 0x100)
            assert_bits(run(h, x, symar.BF16, algo), want)
            assert not h.last_kernel()[0] & CLUSTER
            h.set_variant(algo, 0)
        assert_bits(run(g, x, symar.BF16, symar.LL), want)
        assert g.last_kernel()[0] & CLUSTER                       # the built-in choice for the data+flag protocol
    finally:
        torch.cuda.synchronize()
        h.destroy()
        g.destroy()
