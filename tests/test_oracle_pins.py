"""Pins of the CPU oracle against things other than itself.

Each test fixes one way the oracle could plausibly be wrong: a skipped or
doubled rank, a wrong summation order, a wrong accumulator type, a wrong
rounding mode, a hidden rescale, a broken broadcast of the result.  Expected
values are hand-computed (tests/golden/hand_cases.json), printed by the paper
(tests/golden/paper_values.json), closed forms, or come from an unrelated
library routine (torch CPU elementwise ops, python's exact Fractions).
"""
import json
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import allreduce_oracle as O
from paper_2607_16100_b200 import synth

GOLD = Path(__file__).parent / "golden"


def bf16_bits(values):
    """Exact bf16 bit patterns of numbers that are representable in bf16."""
    w = np.asarray(values, dtype=np.float32).view(np.uint32)
    assert np.all((w & 0xFFFF) == 0), "test value is not a bf16 number"
    return (w >> 16).astype(np.uint16)


def bits_eq(a, b):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    return np.array_equal(a.view(np.uint8), b.view(np.uint8))


def as_wire(rows, dtype):
    if dtype == "f32":
        return np.asarray(rows, dtype=np.float32)
    return np.stack([bf16_bits(r) for r in rows])


# ---- hand-computed cases ----------------------------------------------------

_cases = json.loads((GOLD / "hand_cases.json").read_text())["cases"]


@pytest.mark.parametrize("case", _cases, ids=[c["name"] for c in _cases])
def test_hand_cases(case):
    x = as_wire(case["in"], case["dtype"])
    want = as_wire([case["out"]], case["dtype"])[0]
    out = O.allreduce(x)
    for r in range(x.shape[0]):
        assert bits_eq(out[r], want), (case["name"], r, out[r], want)


# ---- invariants -------------------------------------------------------------

@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
@pytest.mark.parametrize("P", [2, 4, 8])
def test_all_outputs_identical(dtype, dist, P):
    x = synth.make_inputs(dist, dtype, P, 1000, seed=11)
    out = O.allreduce(x)
    for r in range(1, P):
        assert bits_eq(out[r], out[0])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_p1_is_identity(dtype):
    specials = np.array([0.0, -0.0, 1.0, -1.5, 1e-45, -1e-40, 3.0e38, np.inf, -np.inf],
                        dtype=np.float32)
    if dtype == "f32":
        x = specials[None, :]
    else:
        x = (specials.view(np.uint32) >> 16).astype(np.uint16)[None, :]
    out = O.allreduce(x)
    assert bits_eq(out, x)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P", [2, 4, 8])
def test_integer_inputs_sum_exactly(dtype, P):
    # integers in [-8, 8]: every partial sum is at most 64 in magnitude, exact
    # in binary32 and in bf16, so the result is the int64 sum in any order.
    x = synth.make_inputs("int_pm8", dtype, P, 4096, seed=synth.seed_for_config(1))
    xi = (x if dtype == "f32" else synth.bf16_bits_to_f32(x)).astype(np.int64)
    assert xi.min() >= -8 and xi.max() <= 8 and len(np.unique(xi)) == 17
    want = xi.sum(axis=0).astype(np.float32)
    out = O.allreduce(x)
    got = out if dtype == "f32" else synth.bf16_bits_to_f32(out)
    for r in range(P):
        assert np.array_equal(got[r], want)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P", [1, 2, 3, 4, 8])
def test_closed_forms(dtype, P):
    n = 100
    conv = (lambda a: a.astype(np.float32)) if dtype == "f32" else (lambda a: bf16_bits(a))
    back = (lambda a: a) if dtype == "f32" else synth.bf16_bits_to_f32
    # in[q][i] = q + 1  ->  P (P + 1) / 2
    x = np.stack([conv(np.full(n, q + 1.0)) for q in range(P)])
    assert np.all(back(O.allreduce(x)) == P * (P + 1) / 2)
    # in[q][i] = (i mod 17) - 8  ->  P times that
    base = (np.arange(n) % 17 - 8).astype(np.float64)
    x = np.stack([conv(base) for _ in range(P)])
    assert np.array_equal(back(O.allreduce(x))[P - 1], (P * base).astype(np.float32))
    # only rank k is non-zero -> the output is rank k's input, for every k
    src = synth.make_inputs("normal", dtype, 1, n, seed=5)[0]
    for k in range(P):
        x = np.zeros((P, n), dtype=src.dtype)
        x[k] = src
        out = O.allreduce(x)
        for r in range(P):
            assert np.array_equal(back(out[r]), back(src)), (k, r)


@pytest.mark.parametrize("k", [-3, 5])
def test_power_of_two_scaling(k):
    x = synth.make_inputs("uniform", "f32", 8, 2000, seed=3)
    s = np.float32(2.0 ** k)
    assert bits_eq(O.allreduce(x * s), O.allreduce(x) * s)


@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
def test_p2_commutes(dtype, dist):
    x = synth.make_inputs(dist, dtype, 2, 3000, seed=9)
    assert bits_eq(O.allreduce(x), O.allreduce(x[::-1].copy()))


# ---- the error bound the paper states, and its printed constant --------------

def test_gamma_matches_printed_constant():
    paper = json.loads((GOLD / "paper_values.json").read_text())["gamma_63_fp32"]
    g = O.gamma(63)
    # the paper prints two significant digits: 3.8e-6
    assert abs(g - paper["value"]) <= 0.05e-6
    # and the closed form, in exact rational arithmetic
    u = Fraction(1, 2 ** 24)
    assert abs(Fraction(g) - 63 * u / (1 - 63 * u)) < Fraction(1, 10 ** 18)


@pytest.mark.parametrize("P", [2, 4, 8])
def test_fp32_sum_within_forward_error_bound(P):
    x = synth.make_inputs("uniform", "f32", P, 50000, seed=synth.seed_for_config(4))
    got = O.allreduce(x)[0].astype(np.float64)
    exact = O.sum_f64(x)                    # binary64 sum of <= 8 binary32 terms
    bound = O.error_bound(x)
    assert np.all(np.abs(got - exact) <= bound)
    # the bound is not vacuous: rounding does occur somewhere
    assert np.any(got != exact)


@pytest.mark.parametrize("P", [2, 8])
def test_bf16_result_within_half_ulp_of_accumulator(P):
    x = synth.make_inputs("normal", "bf16", P, 50000, seed=synth.seed_for_config(2))
    got = synth.bf16_bits_to_f32(O.allreduce(x)[0]).astype(np.float64)
    exact = O.sum_f64(x)
    # accumulation error (gamma bound) plus one rounding to 8 significand bits
    bound = O.error_bound(x) + 2.0 ** -8 * np.abs(exact) * (1 + 1e-6)
    assert np.all(np.abs(got - exact) <= bound)


# ---- an unrelated library as referee ----------------------------------------

@pytest.mark.parametrize("cfg", ["c1", "c2"])
def test_matches_torch_cpu_elementwise(cfg):
    w = synth.WORKLOADS[cfg]
    x = synth.make_inputs(w["dist"], w["dtype"], w["P"], w["count"], w["seed"])
    if w["dtype"] == "f32":
        t = torch.from_numpy(x)
        acc = t[0].clone()
        for q in range(1, w["P"]):
            acc = acc + t[q]
        want = acc.numpy()
    else:
        t = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16)
        acc = t[0].float()
        for q in range(1, w["P"]):
            acc = acc + t[q].float()
        want = acc.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    out = O.allreduce(x)
    for r in range(w["P"]):
        assert bits_eq(out[r], want)


def test_bf16_narrowing_against_torch_on_all_halfway_patterns():
    # every binary32 whose low 16 bits are 0x7FFF, 0x8000 or 0x8001 around a
    # sample of upper halves: the ties and their neighbours.
    hi = np.arange(0, 0x7F80, 37, dtype=np.uint32)
    words = np.concatenate([(hi << 16) | lo for lo in (0x7FFF, 0x8000, 0x8001, 0x0001, 0xFFFF)])
    words = np.concatenate([words, words | 0x80000000]).astype(np.uint32)
    f = words.view(np.float32)
    want = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([O.narrow_bf16(float(v)) for v in f], dtype=np.uint16)
    finite = np.isfinite(f)
    assert np.array_equal(got[finite], want[finite])


def test_bf16_nan_and_inf():
    assert O.narrow_bf16(float("inf")) == 0x7F80
    assert O.narrow_bf16(float("-inf")) == 0xFF80
    h = O.narrow_bf16(float("nan"))
    assert (h & 0x7F80) == 0x7F80 and (h & 0x007F) != 0
    # overflow of the cut rounds to infinity, as round-to-nearest demands
    big = np.array([0x7F7FFFFF], dtype=np.uint32).view(np.float32)[0]
    assert O.narrow_bf16(float(big)) == 0x7F80
    x = np.array([[0x7F80], [0xFF80]], dtype=np.uint16)       # inf + -inf
    out = O.allreduce(x)
    assert (out[0, 0] & 0x7F80) == 0x7F80 and (out[0, 0] & 0x7F) != 0


def test_widen_is_exact():
    for h in (0x0000, 0x8000, 0x3F80, 0x0001, 0x7F7F, 0xC2F7):
        w = np.array([h << 16], dtype=np.uint32).view(np.float32)[0]
        assert O.widen_bf16(h) == float(w) or (h == 0x8000 and O.widen_bf16(h) == 0.0)


# ---- threaded entry point computes the same bits -----------------------------

@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
def test_threaded_oracle_equals_serial(dtype, dist):
    x = synth.make_inputs(dist, dtype, 8, 100003, seed=21)
    a = O.allreduce(x)
    b, team = O.allreduce_timed_team(x, threads=0)
    assert team >= 1
    assert bits_eq(a, b)


# ---- brute force on tiny inputs with exact rational arithmetic ---------------

def _rn_f32(fr: Fraction) -> np.float32:
    """Correctly rounded binary32 of a rational (python rounds int/int division
    to binary64 correctly; the values used here need < 40 significant bits so
    the second rounding to binary32 cannot double-round incorrectly)."""
    return np.float32(fr.numerator / fr.denominator)


def test_brute_force_small_grid_f32():
    vals = [0.0, 1.0, -1.0, 0.5, -0.5, 2.0 ** -8, -(2.0 ** -8), 256.0, -256.0, 1e8, -1e8]
    rng = np.random.default_rng(7)
    for P in (2, 3, 4):
        picks = rng.integers(0, len(vals), size=(P, 64))
        x = np.array(vals, dtype=np.float32)[picks]
        out = O.allreduce(x)
        for i in range(x.shape[1]):
            acc = Fraction(float(x[0, i]))
            for q in range(1, P):
                acc = Fraction(float(_rn_f32(acc + Fraction(float(x[q, i])))))
            assert float(out[0, i]) == float(acc), (P, i)


# ---- sibling collectives: pinned to the AllReduce oracle and to plain indexing ---------

@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
@pytest.mark.parametrize("P", [1, 2, 4, 8])
def test_allreduce_is_reduce_scatter_then_all_gather(dtype, dist, P):
    # Sec. III: AllReduce decomposes into ReduceScatter and AllGather
    x = synth.make_inputs(dist, dtype, P, P * 37, seed=17)
    assert bits_eq(O.all_gather(O.reduce_scatter(x)), O.allreduce(x))


@pytest.mark.parametrize("dtype,dist", [("f32", "uniform"), ("bf16", "normal")])
@pytest.mark.parametrize("P", [1, 2, 4, 8])
def test_allreduce_is_reduce_then_broadcast(dtype, dist, P):
    x = synth.make_inputs(dist, dtype, P, 101, seed=18)
    red = O.reduce(x)
    assert bits_eq(red, O.allreduce(x)[0])
    for root in range(P):
        y = x.copy()
        y[root] = red
        assert bits_eq(O.broadcast(y, root), O.allreduce(x))


def test_data_movement_collectives_against_numpy_indexing():
    x = synth.make_inputs("normal", "bf16", 4, 50, seed=19)
    ag = O.all_gather(x)
    assert ag.shape == (4, 200)
    for r in range(4):
        assert np.array_equal(ag[r], np.concatenate([x[q] for q in range(4)]))
    for root in range(4):
        assert np.array_equal(O.broadcast(x, root), np.tile(x[root], (4, 1)))


def test_reduce_scatter_hand_case():
    # P = 2, two elements per rank: rank 0 owns columns 0-1, rank 1 columns 2-3
    x = np.array([[1.0, 2.0, 3.0, 4.0], [10.0, 20.0, 30.0, 40.0]], dtype=np.float32)
    out = O.reduce_scatter(x)
    assert np.array_equal(out, np.array([[11.0, 22.0], [33.0, 44.0]], dtype=np.float32))
    # the order pin carries over: chunk sums are rank-ordered binary32 sums
    y = np.array([[1.0] * 4, [1e8] * 4, [-1e8] * 4, [0.0] * 4], dtype=np.float32)
    assert np.all(O.reduce_scatter(y) == 0.0) and np.all(O.reduce(y) == 0.0)
