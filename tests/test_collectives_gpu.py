"""ReduceScatter, AllGather, Broadcast and Reduce on the symmetric heap against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import symar, synth

pytestmark = pytest.mark.gpu

DT = {"f32": symar.F32, "bf16": symar.BF16}
NP = {"f32": np.float32, "bf16": np.uint16}
POISON = 0xA5
OUT = 4 << 20


@pytest.fixture(scope="module")
def heaps():
    hs = {P: symar.SymHeap.on_torch(P, 8 << 20) for P in (1, 2, 4, 8)}
    yield hs
    torch.cuda.synchronize()
    for h in hs.values():
        h.destroy()


def bits(a):
    return np.ascontiguousarray(a).view(np.uint8)


def upload(h, x, off=0):
    for q in range(x.shape[0]):
        h.write_rank(q, off, x[q])


def poison(h, P, nbytes):
    for q in range(P):
        h.write_rank(q, OUT, np.full(nbytes + 64, POISON, dtype=np.uint8))


def fetch(h, P, n, dtype, nbytes_written):
    torch.cuda.synchronize()
    assert h.status()[0] == symar.OK
    out = np.stack([h.read_rank(q, OUT, n, NP[dtype]) for q in range(P)])
    for q in range(P):
        assert np.all(h.read_rank(q, OUT + nbytes_written, 64, np.uint8) == POISON), "wrote past the end"
    return out


COUNTS = [1, 2, 3, 4, 7, 8, 9, 1023, 4096, 10001, 65536]


@pytest.mark.parametrize("n", COUNTS)
@pytest.mark.parametrize("P", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
def test_reduce_scatter(heaps, dtype, dist, P, n):
    h = heaps[P]
    x = synth.make_inputs(dist, dtype, P, P * n, seed=n + P)
    upload(h, x)
    poison(h, P, x.itemsize * n)
    assert h.reduce_scatter(0, OUT, n, DT[dtype]) == symar.OK
    got = fetch(h, P, n, dtype, x.itemsize * n)
    assert np.array_equal(bits(got), bits(O.reduce_scatter(x)))


@pytest.mark.parametrize("n", COUNTS)
@pytest.mark.parametrize("P", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
def test_all_gather(heaps, dtype, dist, P, n):
    h = heaps[P]
    x = synth.make_inputs(dist, dtype, P, n, seed=2 * n + P)
    upload(h, x)
    poison(h, P, x.itemsize * n * P)
    assert h.all_gather(0, OUT, n, DT[dtype]) == symar.OK
    got = fetch(h, P, P * n, dtype, x.itemsize * n * P)
    assert np.array_equal(bits(got), bits(O.all_gather(x)))


@pytest.mark.parametrize("n", [1, 5, 8, 1025, 70001])
@pytest.mark.parametrize("P", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
def test_broadcast_and_reduce_every_root(heaps, dtype, dist, P, n):
    h = heaps[P]
    x = synth.make_inputs(dist, dtype, P, n, seed=3 * n + P)
    upload(h, x)
    nb = x.itemsize * n
    for root in range(P):
        poison(h, P, nb)
        assert h.broadcast(0, OUT, n, DT[dtype], root) == symar.OK
        got = fetch(h, P, n, dtype, nb)
        assert np.array_equal(bits(got), bits(O.broadcast(x, root)))
        poison(h, P, nb)
        assert h.reduce(0, OUT, n, DT[dtype], root) == symar.OK
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        got_root = h.read_rank(root, OUT, n, NP[dtype])
        assert np.array_equal(bits(got_root), bits(O.reduce(x)))
        for q in range(P):                    # non-root outputs stay untouched
            if q != root:
                assert np.all(h.read_rank(q, OUT, nb, np.uint8) == POISON)


def test_allreduce_equals_its_decompositions_on_the_gpu(heaps):
    # Sec. III: ReduceScatter + AllGather and Reduce + Broadcast both rebuild AllReduce
    h = heaps[8]
    n = 8 * 4099
    x = synth.make_inputs("normal", "bf16", 8, n, seed=91)
    upload(h, x)
    mid = 2 << 20
    assert h.reduce_scatter(0, mid, n // 8, symar.BF16) == symar.OK
    assert h.all_gather(mid, OUT, n // 8, symar.BF16) == symar.OK
    torch.cuda.synchronize()
    via_rs_ag = np.stack([h.read_rank(q, OUT, n, np.uint16) for q in range(8)])
    assert h.reduce(0, mid, n, symar.BF16, 3) == symar.OK
    assert h.broadcast(mid, OUT, n, symar.BF16, 3) == symar.OK
    torch.cuda.synchronize()
    via_rd_bc = np.stack([h.read_rank(q, OUT, n, np.uint16) for q in range(8)])
    h.allreduce(0, OUT, n, symar.BF16, symar.AUTO)
    torch.cuda.synchronize()
    direct = np.stack([h.read_rank(q, OUT, n, np.uint16) for q in range(8)])
    want = O.allreduce(x)
    for got in (via_rs_ag, via_rd_bc, direct):
        assert np.array_equal(got, want)
    assert h.status()[0] == symar.OK


def test_collectives_alternate_with_allreduce_in_one_graph(heaps):
    h = heaps[4]
    n = 4 * 2048
    x = synth.make_inputs("uniform", "f32", 4, n, seed=5)
    upload(h, x)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    a, b, c, d = 1 << 20, 2 << 20, 3 << 20, OUT
    with torch.cuda.graph(g, stream=s):
        assert h.reduce_scatter(0, a, n // 4, symar.F32, s.cuda_stream) == symar.OK
        h.allreduce(0, b, n, symar.F32, symar.LL, s.cuda_stream)
        assert h.all_gather(a, c, n // 4, symar.F32, s.cuda_stream) == symar.OK
        h.allreduce(0, d, n, symar.F32, symar.TWOSHOT, s.cuda_stream)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    assert h.status()[0] == symar.OK
    want = O.allreduce(x)
    for off in (b, c, d):
        got = np.stack([h.read_rank(q, off, n, np.float32) for q in range(4)])
        assert np.array_equal(bits(got), bits(want))


def test_collective_argument_errors(heaps):
    h = heaps[4]
    assert h.broadcast(0, OUT, 16, symar.F32, 4) == symar.ERR_INVAL          # root out of range
    assert h.reduce(0, OUT, 16, symar.F32, -1) == symar.ERR_INVAL
    assert h.reduce_scatter(0, 64, 16, symar.F32) == symar.ERR_INVAL         # output overlaps the P-chunk input
    assert h.all_gather(0, 32, 16, symar.F32) == symar.ERR_INVAL             # overlap
    assert h.all_gather(0, OUT, 2 << 20, symar.F32) == symar.ERR_INVAL       # 4 x 8 MiB does not fit
    assert h.reduce_scatter(8, OUT, 16, symar.F32) == symar.ERR_INVAL        # alignment
    assert h.broadcast(0, OUT, 0, symar.F32, 0) == symar.OK                  # no-op
    torch.cuda.synchronize()
    assert h.status()[0] == symar.OK
