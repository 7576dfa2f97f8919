"""The public thread-level buffer primitives (include/symar_llbuffer.cuh; paper Sec. V): a one-shot
AllReduce written only with them (the package's examples/llbuffer_oneshot.cu, after the paper's example
kernel) must give the oracle's bits in both synchronisation modes, over several epochs and launches."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import build, symar, synth

pytestmark = pytest.mark.gpu

LL, SENTINEL = 0, 1


@pytest.fixture(scope="module")
def example():
    lib = ctypes.CDLL(str(build.build_example()))
    fn = lib.llbuffer_oneshot_allreduce
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                   ctypes.c_void_p, ctypes.c_size_t, ctypes.c_size_t, ctypes.c_ulonglong, ctypes.c_int, ctypes.c_int,
                   ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_ulonglong)]
    return fn


@pytest.fixture(scope="module")
def allgather():
    lib = ctypes.CDLL(str(build.build_example()))
    fn = lib.llbuffer_allgather_u64
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p,
                   ctypes.c_size_t, ctypes.c_size_t, ctypes.c_ulonglong, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                   ctypes.c_void_p]
    return fn


class Rig:
    """Input, output and scratch of every rank inside one symmetric heap's user region."""

    def __init__(self, P, mode, ctas, slots):
        self.P, self.mode, self.ctas, self.slots = P, mode, ctas, slots
        self.io_bytes = 1 << 20
        # a CTA's region per epoch holds P rows (one per sender) of `slots` 4-byte elements; two sub-buffers
        self.scratch_bytes = symar.llbuffer_bytes(mode, 4, P * slots, ctas, 2)
        assert self.scratch_bytes == (2 if mode == LL else 1) * 4 * P * slots * ctas * 2
        self.in_off, self.out_off, self.sc_off = 0, self.io_bytes, 2 * self.io_bytes
        self.h = symar.SymHeap.on_torch(P, 2 * self.io_bytes + self.scratch_bytes)
        self.stride = self.h.info().stride
        self.fail = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.epoch = 1
        for q in range(P):
            if mode == SENTINEL:
                symar.llbuffer_init_sentinel(self.h.rank_ptr(q, self.sc_off), self.scratch_bytes)
            else:
                self.h.write_rank(q, self.sc_off, np.zeros(self.scratch_bytes, dtype=np.uint8))
        torch.cuda.synchronize()

    def run(self, fn, x, bf16, threads=128):
        P, count = x.shape
        nwords = x.nbytes // P // 4
        assert x.nbytes // P % 4 == 0
        for q in range(P):
            self.h.write_rank(q, self.in_off, x[q])
            self.h.write_rank(q, self.out_off, np.full(nwords * 4 + 64, 0xA5, dtype=np.uint8))
        used = ctypes.c_ulonglong(0)
        rc = fn(self.mode, P, 1 if bf16 else 0, self.h.rank_ptr(0, self.in_off), self.h.rank_ptr(0, self.out_off),
                self.stride, self.h.rank_ptr(0, self.sc_off), self.stride, nwords, self.epoch, self.ctas, threads,
                self.slots, self.fail.data_ptr(), 0, ctypes.byref(used))
        assert rc == 0
        torch.cuda.synchronize()
        assert int(self.fail.item()) == 0, "a bounded wait ran out"
        self.epoch += used.value
        dt = np.uint16 if bf16 else np.float32
        out = np.stack([self.h.read_rank(q, self.out_off, count, dt) for q in range(P)])
        for q in range(P):
            assert np.all(self.h.read_rank(q, self.out_off + nwords * 4, 64, np.uint8) == 0xA5)
        return out

    def close(self):
        torch.cuda.synchronize()
        self.h.destroy()


@pytest.mark.parametrize("mode", [LL, SENTINEL])
@pytest.mark.parametrize("P", [1, 2, 4, 8])
def test_oneshot_on_the_primitives_matches_the_oracle(example, mode, P):
    rig = Rig(P, mode, ctas=4, slots=256)
    try:
        # sizes below, at and far above one epoch's capacity (4 CTAs x 256 words): 1 to 20 epochs per launch
        for launch, count in enumerate((4, 1024, 1000, 5000, 20480, 3, 4096)):
            x = synth.make_inputs("uniform", "f32", P, count, seed=300 + launch)
            got = rig.run(example, x, bf16=False)
            assert np.array_equal(got.view(np.uint32), O.allreduce(x).view(np.uint32)), (mode, P, count)
        for launch, count in enumerate((8, 2048, 30000)):
            x = synth.make_inputs("normal", "bf16", P, count, seed=400 + launch)
            got = rig.run(example, x, bf16=True, threads=64)
            assert np.array_equal(got, O.allreduce(x)), (mode, P, count)
    finally:
        rig.close()


def test_sentinel_valued_payload_and_flag_wrap(example):
    # a payload word equal to the sentinel (all ones, a NaN) is sent with its lowest bit cleared: still a NaN
    rig = Rig(2, SENTINEL, ctas=2, slots=64)
    try:
        x = synth.make_inputs("uniform", "f32", 2, 256, seed=1)
        x.view(np.uint32)[0, 5] = 0xFFFFFFFF
        got = rig.run(example, x, bf16=False)
        want = O.allreduce(x)
        assert np.isnan(got[0, 5]) and np.isnan(got[1, 5])
        keep = np.ones(256, dtype=bool)
        keep[5] = False
        assert np.array_equal(got[:, keep].view(np.uint32), want[:, keep].view(np.uint32))
    finally:
        rig.close()
    # LL: epochs around the 32-bit flag wrap (the flag value 0 is skipped, sub-buffers keep alternating)
    rig = Rig(4, LL, ctas=2, slots=128)
    try:
        rig.epoch = (1 << 32) - 3
        for launch in range(4):
            x = synth.make_inputs("uniform", "f32", 4, 700, seed=launch)     # 3 epochs per launch
            got = rig.run(example, x, bf16=False)
            assert np.array_equal(got.view(np.uint32), O.allreduce(x).view(np.uint32)), launch
        assert rig.epoch > (1 << 32)
    finally:
        rig.close()


def test_size_helper_rejects_bad_arguments():
    assert symar.llbuffer_bytes(LL, 4, 100, 3, 2) == 2 * 4 * 100 * 3 * 2
    assert symar.llbuffer_bytes(SENTINEL, 8, 100, 3, 0) == 8 * 100 * 3
    assert symar.llbuffer_bytes(2, 4, 100, 3, 2) == 0
    assert symar.llbuffer_bytes(LL, 3, 100, 3, 2) == 0
    assert symar.llbuffer_bytes(LL, 4, 100, 0, 2) == 0


@pytest.mark.parametrize("mode", [LL, SENTINEL])
@pytest.mark.parametrize("P", [2, 8])
def test_allgather_of_64_bit_words_on_the_primitives(allgather, mode, P):
    # 8-byte elements (16-byte LL slots), send / recv / reset one at a time, an undivided buffer
    ctas, nwords = 3, 1000
    per_cta = (nwords + ctas - 1) // ctas
    scratch = symar.llbuffer_bytes(mode, 8, P * per_cta, ctas, 0)
    assert scratch == (2 if mode == LL else 1) * 8 * P * per_cta * ctas
    io = 1 << 17
    h = symar.SymHeap.on_torch(P, 2 * io + scratch)
    fail = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        stride = h.info().stride
        for q in range(P):
            if mode == SENTINEL:
                symar.llbuffer_init_sentinel(h.rank_ptr(q, 2 * io), scratch)
            else:
                h.write_rank(q, 2 * io, np.zeros(scratch, dtype=np.uint8))
        rng = np.random.default_rng(5)
        for launch in range(3):                                  # the undivided region is reused every launch
            x = rng.integers(0, 1 << 63, size=(P, nwords), dtype=np.uint64)
            x[0, 7] = np.uint64(0xFFFFFFFFFFFFFFFF) if mode == LL else x[0, 7]      # all ones is fine for LL
            for q in range(P):
                h.write_rank(q, 0, x[q])
            rc = allgather(mode, P, h.rank_ptr(0, 0), h.rank_ptr(0, io), stride, h.rank_ptr(0, 2 * io), stride, nwords,
                           launch + 1, ctas, 128, fail.data_ptr(), 0)
            assert rc == 0
            torch.cuda.synchronize()
            assert int(fail.item()) == 0
            for q in range(P):
                got = h.read_rank(q, io, P * nwords, np.uint64)
                assert np.array_equal(got, x.reshape(-1)), (mode, P, launch, q)
    finally:
        torch.cuda.synchronize()
        h.destroy()


@pytest.mark.parametrize("P,ctas,slots,epochs", [(2, 8, 128, 4000), (8, 4, 64, 1500), (4, 16, 32, 2500)])
def test_16_byte_slots_of_64_bit_elements_are_observed_whole(P, ctas, slots, epochs):
    # An 8-byte element travels as {payload64, flag64} in ONE 16-byte store; the buffer is correct only if a
    # reader never sees the new flag beside the old payload.  Thousands of epochs in one launch, every payload
    # spelling out its epoch, sender and slot, seeded idle times shifting which rank is ahead: no payload may
    # disagree with its flag, and no wait may run out.
    lib = ctypes.CDLL(str(build.build_example()))
    fn = lib.llbuffer_slot_stress_u64
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.c_ulonglong,
                   ctypes.c_uint, ctypes.c_uint, ctypes.c_uint, ctypes.c_void_p, ctypes.c_void_p]
    nbytes = symar.llbuffer_bytes(LL, 8, P * slots, ctas, 2)
    assert nbytes == 2 * 8 * P * slots * ctas * 2
    h = symar.SymHeap.on_torch(P, nbytes)
    try:
        for q in range(P):
            h.write_rank(q, 0, np.zeros(nbytes, dtype=np.uint8))
        epoch = 1
        for seed, idle_ns in ((1, 0), (2, 2000), (3, 300), (4, 20000)):
            counts = torch.zeros(3, dtype=torch.int64, device="cuda")
            n = epochs if idle_ns <= 2000 else epochs // 10
            assert fn(P, h.rank_ptr(0, 0), h.info().stride, ctas, slots, epoch, n, seed, idle_ns, counts.data_ptr(), 0) == 0
            torch.cuda.synchronize()
            timeouts, mismatches, checked = (int(v) for v in counts.cpu())
            assert timeouts == 0 and mismatches == 0, (seed, timeouts, mismatches)
            assert checked == P * ctas * slots * (P - 1) * n
            epoch += n
    finally:
        torch.cuda.synchronize()
        h.destroy()
