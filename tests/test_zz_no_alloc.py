"""allreduce_static(): the entry point for callers that cannot allocate device
memory (frozen memory pool, plugin without an allocator, a deployment that fixes
all device memory at start-up).  It keeps its LL scratch in a static device array
inside the library, so the caller brings only inputs and outputs.

The check: through the C ABI, on calls in a row, its output must equal the CPU
oracle's bit for bit, and the output of the existing heap-based allreduce() (the
tolerance all parity tests here use).  The calls differ in rank count, dtype,
size and data, so anything the shared static array kept from an earlier call
would show.  Free device memory must not move across a call.  The file sorts
last so that a run stopping at the first failure has already run every other
test; it passes alone in a fresh process as well.
"""
import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import symar, synth

pytestmark = pytest.mark.gpu

NP_DT = {symar.F32: np.float32, symar.BF16: np.uint16}
TORCH_DT = {symar.F32: torch.float32, symar.BF16: torch.int16}


def heap_result(P, x, dtype):
    """The existing entry point: symmetric heap + allreduce()."""
    count = x.shape[1]
    h = symar.SymHeap.on_torch(P, 1 << 20)
    try:
        for q in range(P):
            h.write_rank(q, 0, x[q])
        h.allreduce(0, 1 << 19, count, dtype, symar.LL)
        torch.cuda.synchronize()
        assert h.status()[0] == symar.OK
        return np.stack([h.read_rank(q, 1 << 19, count, NP_DT[dtype]) for q in range(P)])
    finally:
        h.destroy()


def static_result(P, x, dtype, pitch_elems, stream=0):
    """The new entry point on plain torch buffers."""
    count = x.shape[1]
    es = symar.DTYPE_SIZE[dtype]
    host = np.zeros((P, pitch_elems), dtype=NP_DT[dtype])
    host[:, :count] = x
    tin = torch.from_numpy(host.view(np.int16) if dtype == symar.BF16 else host).cuda()
    tout = torch.full_like(tin, 0x5A5A if dtype == symar.BF16 else 12345.0)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    rc = symar.allreduce_static(tin.data_ptr(), tout.data_ptr(), pitch_elems * es, P, count, dtype,
                                status.data_ptr(), stream)
    assert rc == symar.OK
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status must be cleared and stay clear"
    out = tout.cpu().numpy()
    if dtype == symar.BF16:
        out = out.view(np.uint16)
    # nothing beyond the message may be written
    guard = 0x5A5A if dtype == symar.BF16 else np.float32(12345.0)
    assert np.all(out[:, count:] == guard)
    return out[:, :count].copy()


def test_static_entry_point_matches_oracle_and_heap_entry_point_on_calls_in_a_row():
    # call 1: P = 8, bf16, the 16 KiB decode-step message
    x1 = synth.make_inputs("normal", "bf16", 8, 8192, seed=synth.seed_for_config(2))
    got1 = static_result(8, x1, symar.BF16, pitch_elems=8192 + 64)
    # call 2, straight after: other rank count, dtype, ragged size, other data
    x2 = synth.make_inputs("uniform", "f32", 4, 5003, seed=99)
    got2 = static_result(4, x2, symar.F32, pitch_elems=5008)
    # calls 3 and 4: a single rank (a copy) and two ranks, between the eight-rank calls
    x3 = synth.make_inputs("normal", "bf16", 1, 777, seed=5)
    got3 = static_result(1, x3, symar.BF16, pitch_elems=784)
    x4 = synth.make_inputs("uniform", "f32", 2, 8192, seed=6)
    got4 = static_result(2, x4, symar.F32, pitch_elems=8192)
    # call 5: the first shape again with new data (scratch rows are reused)
    x5 = synth.make_inputs("normal", "bf16", 8, 8192, seed=1234)
    got5 = static_result(8, x5, symar.BF16, pitch_elems=8192)
    for got, x, P, dt in ((got1, x1, 8, symar.BF16), (got2, x2, 4, symar.F32), (got3, x3, 1, symar.BF16),
                          (got4, x4, 2, symar.F32), (got5, x5, 8, symar.BF16)):
        want = O.allreduce(x)                               # the definition, on the CPU
        assert np.array_equal(got.view(np.uint8), want.view(np.uint8)), (P, dt)
        assert np.array_equal(got.view(np.uint8), heap_result(P, x, dt).view(np.uint8)), (P, dt)


def test_static_entry_point_leaves_free_device_memory_alone():
    x = synth.make_inputs("normal", "bf16", 8, 4096, seed=11)
    static_result(8, x, symar.BF16, pitch_elems=4096)        # the first call on the device does the set-up
    tin = torch.from_numpy(x.view(np.int16)).cuda()
    tout = torch.zeros_like(tin)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        assert symar.allreduce_static(tin.data_ptr(), tout.data_ptr(), 4096 * 2, 8, 4096, symar.BF16) == symar.OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert np.array_equal(tout.cpu().numpy().view(np.uint16), O.allreduce(x))


def test_static_entry_point_limits_and_arguments():
    buf = torch.zeros(1 << 16, dtype=torch.float32, device="cuda")
    p = buf.data_ptr()
    half = p + (1 << 17)
    big = symar.STATIC_MAX_BYTES // 4 + 1
    assert symar.allreduce_static(p, half, 1 << 16, 2, big, symar.F32) == symar.ERR_UNSUPPORTED
    assert symar.allreduce_static(p, half, 1 << 12, 3, 16, symar.F32) == symar.ERR_INVAL        # rank count
    assert symar.allreduce_static(p + 4, half, 1 << 12, 2, 16, symar.F32) == symar.ERR_INVAL    # alignment
    assert symar.allreduce_static(p, half, 40, 2, 16, symar.F32) == symar.ERR_INVAL             # pitch not 16-byte aligned
    assert symar.allreduce_static(p, half, 48, 2, 16, symar.F32) == symar.ERR_INVAL             # pitch below the 64-byte row
    assert symar.allreduce_static(p, p + 64, 1 << 12, 2, 64, symar.F32) == symar.ERR_INVAL      # overlap
    assert symar.allreduce_static(0, half, 1 << 12, 2, 16, symar.F32) == symar.ERR_INVAL
    assert symar.allreduce_static(p, half, 1 << 12, 2, 0, symar.F32) == symar.OK                # no-op
    torch.cuda.synchronize()
