#!/usr/bin/env python
"""Benchmark of the barrier-free symmetric-memory AllReduce on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--out-dir DIR]

ONE short JSON line on stdout (rank 0), fewer than 2000 characters.  A "step" is one AllReduce of
the bandwidth workload: P = 8 emulated ranks, fp32, 64 Mi elements (256 MiB) per rank, inputs
U(-1, 1), two-shot algorithm.  `value` is algorithmic bytes (every input byte read once + every
output byte written once = 2 P M) per second with the inputs resident in HBM.  The latency half of
the metric (P = 8, bf16, 16 KiB per rank, p50 against the speed-of-light bound measured in the same
process) and the 160-call decode-step graph ride in the same line as a handful of numbers under
`latency_16KB` and `decode_trace`.

Everything else -- per-algorithm rows, the 16 KiB..1 MiB sweep with the selector's choice, the
sampled flag round trips, phase stamps, the tuner's table, the context measurements -- goes to one
file per workload in the directory given by --out-dir: results_c2.json, results_c3.json, results_c4.json,
results_c5.json.  The line names them under `details`.

N > 1 runs N independent replicas (one process and one heap per GPU; the path itself is a
single-GPU emulation and has no exchange between GPUs).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "p50 AllReduce latency µs @16KB vs SoL; HBM GB/s @256MB (8 emulated ranks)"
L2_BYTES = 126 << 20


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ---------------------------------------------------------------------------------
# clocks: nvidia-smi sampled in the background during a timed region
# ---------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._pump, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        rows = [l for (t, l) in self.lines if t_begin <= t <= t_end + 0.02] or \
            [l for (t, l) in self.lines if t_begin <= t <= t_end + 0.2] or [l for (_, l) in self.lines]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------
# multi-process plumbing (replicas only: no data-path collective)
# ---------------------------------------------------------------------------------
def max_over_ranks(dist, ms: float, device) -> float:
    """Slowest rank's time: the job is as slow as its slowest replica."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_step: float, world: int, steps: int, total_ms: float) -> float:
    """Aggregate throughput: every replica processed the same units in `total_ms`."""
    return units_per_rank_step * world * steps / (total_ms * 1e-3)


# ---------------------------------------------------------------------------------
# reference arm: the CPU oracle on the host cores
# ---------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import allreduce_oracle as O
    from paper_2607_16100_b200 import synth
    w = synth.WORKLOADS["c4"]
    P = w["P"]
    sample = 8 << 20                      # elements per rank per step: 1/8 of the workload
    x = synth.make_inputs(w["dist"], w["dtype"], P, sample, w["seed"])
    team = 1
    for _ in range(max(1, args.warmup)):
        _, team = O.allreduce_timed_team(x, threads=0)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.allreduce_timed_team(x, threads=0)
    dt = time.perf_counter() - t0
    algbytes = 2 * P * sample * 4
    gbs = algbytes * args.steps / dt / 1e9
    desc = f"{sample} of {w['count']} elements per rank per step (1/8 of the workload), all host cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "c4: P=8 emulated ranks, fp32, 64Mi elements (256 MiB) per rank, U(-1,1)",
                   "sample": desc},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": team, "kind": "oracle", "sample": desc},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------
# latency harness: K calls in one CUDA graph, one replay = one sample
# ---------------------------------------------------------------------------------
def graph_of(torch, stream, enqueue, K):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for k in range(K):
            enqueue(k, stream.cuda_stream)
    return g


def time_graph(torch, g, stream, K, reps, warm=10):
    with torch.cuda.stream(stream):
        for _ in range(warm):
            g.replay()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in ev:
            a.record(stream)
            g.replay()
            b.record(stream)
    stream.synchronize()
    us = np.array([a.elapsed_time(b) for a, b in ev]) * 1000.0 / K
    return {"p10": float(np.percentile(us, 10)), "p50": float(np.percentile(us, 50)),
            "p90": float(np.percentile(us, 90))}


def time_stream(torch, stream, enqueue, n, warm=50):
    """Stream-launched (no graph) per-call p50: events around blocks of 20 calls."""
    with torch.cuda.stream(stream):
        for k in range(warm):
            enqueue(k, stream.cuda_stream)
        blocks = []
        for _ in range(n // 20):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for k in range(20):
                enqueue(k, stream.cuda_stream)
            b.record(stream)
            blocks.append((a, b))
    stream.synchronize()
    us = np.array([a.elapsed_time(b) for a, b in blocks]) * 1000.0 / 20
    return float(np.percentile(us, 50))


def sample_flag_round_trips(torch, symar):
    """The flag round trip depends on which SMs the two CTAs sit on (measured: mostly on the one
    that sends first; 0.5-0.7 us from some SMs, 0.9-1.1 us from others), and the ranks of the
    AllReduce are spread over the whole chip.  Sample pairs with both ends spread over a
    one-CTA-per-SM launch; the bound uses the median pair, min and max are reported."""
    pairs = []
    nsm = torch.cuda.get_device_properties(0).multi_processor_count
    firsts = [int(round(i * (nsm - 1) / 11)) for i in range(12)]
    for i, first in enumerate(firsts):
        for off in (1, nsm // 3 + i, nsm // 2 + 2 * i + 1):
            partner = (first + off) % nsm
            if partner == first:
                continue
            try:
                ns, sm = symar.probe_pingpong_blocks(first, partner, nsm, 5000)
                pairs.append({"first_block": first, "partner_block": partner, "smids": list(sm),
                              "round_trip_us": ns / 1000.0})
            except symar.SymarError:
                pass
    rts = sorted(p["round_trip_us"] for p in pairs)
    nan = float("nan")
    return {"min_us": rts[0] if rts else nan, "median_us": rts[len(rts) // 2] if rts else nan,
            "max_us": rts[-1] if rts else nan, "pairs": pairs}


def spread(values):
    v = [x for x in values if x == x]
    if not v:
        return {"median": None, "min": None, "max": None, "n": 0}
    return {"median": float(np.median(v)), "min": float(min(v)), "max": float(max(v)), "n": len(v)}


def oracle_us(O, x):
    """The CPU oracle on one message, in microseconds: single thread and all host cores (best of 5)."""
    one = all_ = 1e30
    team = 1
    for _ in range(5):
        t0 = time.perf_counter()
        O.allreduce_timed_team(x, threads=1)
        one = min(one, time.perf_counter() - t0)
        t0 = time.perf_counter()
        _, team = O.allreduce_timed_team(x, threads=0)
        all_ = min(all_, time.perf_counter() - t0)
    return {"single_thread_us": one * 1e6, "all_cores_us": all_ * 1e6, "cores": team}


def sys_scope_numbers(shapes, quick):
    """16 KiB one-shot and LL from the build whose flags, signals and data+flag accesses are at
    system scope (what an NVLink domain needs), in a child process that loads that library."""
    try:
        from paper_2607_16100_b200 import build as B
        lib = B.build_lib_sys()
        env = dict(os.environ, SYMAR_LIB=str(lib))
        r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--scope-probe", json.dumps(shapes)] +
                           (["--quick"] if quick else []), capture_output=True, text=True, env=env, timeout=300)
        if r.returncode != 0:
            return {"error": (r.stderr or r.stdout)[-300:]}
        return json.loads(r.stdout.strip().splitlines()[-1])
    except Exception as exc:
        return {"error": f"{type(exc).__name__}: {exc}"}


def scope_probe(shapes_json, quick):
    """Child of sys_scope_numbers(): times the given (algorithm, variant, shape) rows at 16 KiB, P = 8."""
    import torch
    from oracle import allreduce_oracle as O
    from paper_2607_16100_b200 import symar, synth
    shapes = json.loads(shapes_json)
    stream = torch.cuda.Stream()
    P, count, out_off = 8, 8192, 1 << 20
    h = symar.SymHeap.on_torch(P, 2 << 20)
    x = synth.make_inputs("normal", "bf16", P, count, synth.seed_for_config(2))
    for q in range(P):
        h.write_rank(q, 0, x[q])
    want = O.allreduce(x)
    out = {"library": str(symar.LIB_PATH.name)}
    for name, (algo, variant, ctas, threads) in shapes.items():
        h.set_variant(algo, variant if variant else 1 << 31)
        h.set_launch(algo, ctas, threads)
        enq = lambda k, s: h.allreduce(0, out_off, count, symar.BF16, algo, s)
        enq(0, stream.cuda_stream)
        stream.synchronize()
        got = np.stack([h.read_rank(q, out_off, count, np.uint16) for q in range(P)])
        g = graph_of(torch, stream, enq, 64)
        r = time_graph(torch, g, stream, 64, 60 if quick else 200)
        out[name] = {"p50_us": r["p50"], "bit_exact": bool(np.array_equal(got, want)) and h.status()[0] == 0}
        h.set_variant(algo, 0)
        h.set_launch(algo, 0, 0)
    h.destroy()
    print(json.dumps(out))


def run_case(spec, steps, warmup):
    """`--case ALGO:BYTES[:P[:VARIANT[:CTAS:THREADS]]]` (or `--case c1`): a few stream-launched calls of ONE
    algorithm on a bf16 message of BYTES per rank, checked against the oracle -- a small, self-ending command for
    profilers (a few MiB on the device, `warmup` + `steps` launches)."""
    import torch
    from oracle import allreduce_oracle as O
    from paper_2607_16100_b200 import symar, synth
    if spec == "c1":          # the smallest workload as it is defined: P = 4, fp32, 1024 integer-valued elements, one-shot
        w = synth.WORKLOADS["c1"]
        algo, P, variant, ctas, threads = symar.ONESHOT, w["P"], 0, 0, 0
        count, nbytes, dt, npdt = w["count"], w["count"] * 4, symar.F32, np.uint32
        x = synth.make_inputs(w["dist"], "f32", P, count, w["seed"])
    else:
        f = spec.split(":")
        algo = {v: k for k, v in symar.ALGO_NAMES.items()}[f[0]]
        nbytes = int(f[1])
        P = int(f[2]) if len(f) > 2 else 8
        variant = int(f[3], 0) if len(f) > 3 else 0
        ctas, threads = (int(f[4]), int(f[5])) if len(f) > 5 else (0, 0)
        count, dt, npdt = nbytes // 2, symar.BF16, np.uint16
        x = synth.make_inputs("normal", "bf16", P, count, synth.seed_for_config(2))
    out_off = (nbytes + 4095) // 4096 * 4096
    h = symar.SymHeap.on_torch(P, max(2 * out_off, 1 << 16))
    for q in range(P):
        h.write_rank(q, 0, x[q])
    if variant:
        h.set_variant(algo, variant)
    if ctas or threads:
        h.set_launch(algo, ctas, threads)
    stream = torch.cuda.Stream()
    call = lambda: h.allreduce(0, out_off, count, dt, algo, stream.cuda_stream)
    for _ in range(max(1, warmup)):
        call()
    stream.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        a.record(stream)
        for _ in range(steps):
            call()
        b.record(stream)
    stream.synchronize()
    got = np.stack([h.read_rank(q, out_off, count, npdt) for q in range(P)])
    al, c, t = h.last_choice()
    print(json.dumps({"case": spec, "algo": symar.ALGO_NAMES[al], "ctas_per_rank": c, "threads": t,
                      "variant": h.last_kernel()[0], "launches": max(1, warmup) + steps,
                      "stream_launched_us_per_call": a.elapsed_time(b) * 1000.0 / steps,
                      "bit_exact": bool(np.array_equal(got, O.allreduce(x).view(npdt))) and h.status()[0] == 0}))
    h.destroy()


def latency_suite(torch, symar, synth, hbm_gbs, quick=False, autotune=True):
    """C2 (16 KiB vs SoL), C3 (sweep + selector), C5 (decode-step graph)."""
    from oracle import allreduce_oracle as O
    out = {}
    stream = torch.cuda.Stream()
    K, reps = 64, (60 if quick else 300)
    REPEATS = 3 if quick else 5
    names = dict(symar.ALGO_NAMES)
    ALL = (symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL,
           symar.AUTO)

    # speed-of-light parts (paper Sec. VI), measured here
    fence_ns = symar.probe_fence(20000)
    rt0 = sample_flag_round_trips(torch, symar)
    rt_ns, rt_min_ns = 1000.0 * rt0["median_us"], 1000.0 * rt0["min_us"]
    out["flag_round_trip_pairs"] = rt0
    bytes_us = lambda nbytes, P_: 2 * P_ * nbytes / (hbm_gbs * 1e9) * 1e6      # "bytes at peak": the measured copy rate

    # the barrier that the method removes (Sec. III-B), for context: P CTAs, all signal all, all wait for all
    try:
        out["barrier_us"] = {f"P{p_}": {"relaxed": symar.probe_barrier(p_, 3000, False) / 1e3,
                                         "release_acquire": symar.probe_barrier(p_, 3000, True) / 1e3}
                             for p_ in (2, 4, 8)}
    except symar.SymarError as exc:
        out["barrier_us"] = {"error": str(exc)}

    def empty_floor(cx, py, T, pdl=True, n=None):
        """The launch floor of a grid (cx, py) of T threads: an empty kernel, with programmatic dependent launch
        as the library launches; the smaller of the plain launch and the launch with each column's py CTAs as
        one thread-block cluster (the library uses either, and the cluster launch is often the cheaper one)."""
        probe = symar.probe_empty_pdl if pdl else symar.probe_empty
        g = graph_of(torch, stream, lambda k, s: probe(cx, py, T, s), K)
        r = time_graph(torch, g, stream, K, n or reps)
        r["form"] = "plain"
        if pdl and 2 <= py <= 8:
            c_ = empty_floor_cluster(cx, py, T, n)
            r["plain_p50"], r["slot_clusters_p50"] = r["p50"], c_
            if c_ is not None and c_ < r["p50"]:
                r["p50"], r["form"] = c_, "slot clusters"
        return r

    def empty_floor_cluster(cx, py, T, n=None):
        try:
            g = graph_of(torch, stream, lambda k, s: symar.probe_empty_cluster(cx, py, T, s), K)
            return time_graph(torch, g, stream, K, n or reps)["p50"]
        except symar.SymarError:
            return None               # such a cluster cannot be launched

    for P in (8, 4):
        h = symar.SymHeap.on_torch(P, 24 << 20)
        t0 = time.time()
        if autotune:
            h.autotune(symar.BF16)
        tune_s = time.time() - t0
        out_off = 12 << 20
        res = {"autotune_seconds": tune_s}
        if autotune:
            # what the tuner measured (graphs of back-to-back calls, warm): per size the time of every
            # bit-reproducible algorithm at its best shape -- the selector's whole landscape
            table = []
            for log2 in range(5, 24):
                us = {}
                for a_ in (symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL, symar.TWOSHOT_LL,
                           symar.TWOSHOT_SENTINEL):
                    e_ = h.tuned_entry(symar.BF16, log2, a_)
                    if e_ and e_[0] > 0 and e_[2] < 1e29:
                        us[names[a_]] = round(e_[2], 3)
                if us:
                    table.append({"bytes_per_rank": 1 << log2, "us": us, "best": min(us, key=us.get)})
            out.setdefault("tuner_table_bf16", {})[f"P{P}"] = table

        def load_inputs(count, heap=None):
            x = synth.make_inputs("normal", "bf16", P, count, synth.seed_for_config(2))
            for q in range(P):
                (heap or h).write_rank(q, 0, x[q])
            return x

        def untuned_default(count, n=None):
            """The same call on a heap that was never tuned: the built-in algorithm and launch shape."""
            hu = symar.SymHeap.on_torch(P, 24 << 20)
            try:
                x = load_inputs(count, hu)
                enq = lambda k, s: hu.allreduce(0, out_off, count, symar.BF16, symar.AUTO, s)
                enq(0, stream.cuda_stream)
                stream.synchronize()
                a, c, t = hu.last_choice()
                got = np.stack([hu.read_rank(q, out_off, count, np.uint16) for q in range(P)])
                exact = bool(np.array_equal(got, O.allreduce(x))) and hu.status()[0] == 0
                r = time_graph(torch, graph_of(torch, stream, enq, K), stream, K, n or reps)
                return {"p50_us": r["p50"], "algo": names[a], "shape": [c, t], "variant": hu.last_kernel()[0],
                        "bit_exact": exact}
            finally:
                stream.synchronize()
                hu.destroy()

        def bench_size(count, algos, stream_too=False, n=None):
            x = load_inputs(count)
            want = O.allreduce(x)
            row = {}
            for algo in algos:
                enq = lambda k, s, algo=algo: h.allreduce(0, out_off, count, symar.BF16, algo, s)
                enq(0, stream.cuda_stream)
                stream.synchronize()
                a, c, t = h.last_choice()
                got = np.stack([h.read_rank(q, out_off, count, np.uint16) for q in range(P)])
                exact = bool(np.array_equal(got, want)) and h.status()[0] == 0
                g = graph_of(torch, stream, enq, K)
                r = time_graph(torch, g, stream, K, n or reps)
                r.update({"algo": names[a], "ctas_per_rank": c, "threads": t, "variant": h.last_kernel()[0],
                          "bit_exact": exact})
                if algo == symar.TWOSHOT_ATOMIC:
                    # order of the atomic adds is free: all ranks identical, values within one bf16 ulp
                    # of the oracle plus 1e-6 * sum|x| (bit_exact is reported as seen, not required)
                    wide = lambda a_: (a_.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
                    gw, ww = wide(got[0]), wide(want[0])
                    tol = 1e-6 * np.abs(wide(x)).sum(axis=0) + \
                        2.0 ** (np.floor(np.log2(np.maximum(np.abs(ww), 1e-30))) - 7)
                    r["within_tolerance"] = bool(np.all(np.abs(gw - ww) <= tol)) and \
                        all(np.array_equal(got[q], got[0]) for q in range(1, P)) and h.status()[0] == 0
                if stream_too:
                    r["stream_launched_p50"] = time_stream(torch, stream, enq, 400)
                row[names[algo]] = r
            return row

        def with_variant(algo, variant, ctas, threads, count=8192):
            """One row of `algo` with the given variant bits and launch shape."""
            h.set_launch(algo, ctas, threads)
            h.set_variant(algo, variant if variant else 1 << 31)
            try:
                return bench_size(count, (algo,))[names[algo]]
            finally:
                h.set_variant(algo, 0)
                h.set_launch(algo, 0, 0)

        # C2: 16 KiB per rank
        if P == 8:
            row = bench_size(8192, ALL, stream_too=True)
            best = min(row.values(), key=lambda r: r["p50"])
            floor = empty_floor(best["ctas_per_rank"], P, best["threads"])
            floor11 = empty_floor(1, 1, 1)
            t_bytes_us = bytes_us(16384, P)
            sol = floor["p50"] + rt_ns / 1000.0 + t_bytes_us
            # the whole comparison again, bound and kernel interleaved in this process, REPEATS times; the
            # bound then uses the SMALLEST empty launch seen (it is a floor; its p50 wanders between 0.50
            # and 0.73 us from one measurement to the next) and the median of the pair medians
            rep_rows = [{"p50_us": best["p50"], "empty_launch_us": floor["p50"],
                         "flag_round_trip_median_us": rt0["median_us"], "flag_round_trip_min_us": rt0["min_us"]}]
            for _ in range(REPEATS):
                rt_i = sample_flag_round_trips(torch, symar)
                fl_i = empty_floor(best["ctas_per_rank"], P, best["threads"])["p50"]
                p_i = bench_size(8192, (symar.AUTO,))["auto"]["p50"]
                rep_rows.append({"p50_us": p_i, "empty_launch_us": fl_i, "flag_round_trip_median_us": rt_i["median_us"],
                                 "flag_round_trip_min_us": rt_i["min_us"]})
            floor_us = min(r_["empty_launch_us"] for r_ in rep_rows)
            rt_us = float(np.median([r_["flag_round_trip_median_us"] for r_ in rep_rows]))
            rt_min_us = min(r_["flag_round_trip_min_us"] for r_ in rep_rows)
            sol = floor_us + rt_us + t_bytes_us
            sol_fast = floor_us + rt_min_us + t_bytes_us
            for r_ in rep_rows:
                r_["ratio_to_sol"] = r_["p50_us"] / sol
            p50_all = spread([r_["p50_us"] for r_ in rep_rows])
            # the same call with every reader on copy 0 of the flags and counters (no placement on the L2 halves)
            h.set_placement(False)
            unplaced = bench_size(8192, (symar.AUTO,))["auto"]
            h.set_placement(True)
            o_a, o_c, o_t = h.query_choice(8192, symar.BF16, symar.ONESHOT)
            o_var = row["oneshot"]["variant"]
            release = with_variant(symar.ONESHOT, o_var | 0x8000, o_c, o_t)
            prior = with_variant(symar.ONESHOT, 0x4000 | 0x100, o_c, o_t)
            phases = {}
            for a_ in (symar.ONESHOT, symar.LL, symar.TWOSHOT):
                try:
                    load_inputs(8192)
                    ph = [h.debug_phases(0, out_off, 8192, symar.BF16, a_) for _ in range(31)]
                    phases[names[a_]] = {str(k): {f: float(np.median([p_[k][f] for p_ in ph])) / 1e3
                                                  for f in ("first", "mean", "last")} for k in sorted(ph[0])}
                except symar.SymarError as exc:
                    phases[names[a_]] = {"error": str(exc)}
            l_var = row["ll"]["variant"]
            sys_scope = sys_scope_numbers(
                {"oneshot": [symar.ONESHOT, o_var, o_c, o_t],
                 "oneshot_release_signal": [symar.ONESHOT, o_var | 0x8000, o_c, o_t],
                 "ll": [symar.LL, l_var, row["ll"]["ctas_per_rank"], row["ll"]["threads"]]}, quick)
            out["latency_16KB"] = {
                "workload": "c2: P=8, bf16, 8192 elements (16 KiB) per rank, N(0,1); buffers L2-resident (warm)",
                "harness": f"{K} back-to-back calls in one CUDA graph, one replay = one sample, {reps} samples; "
                           "numerator and denominator use the same harness",
                "p50_us": p50_all["median"], "best": best, "per_algo": row,
                "repeats": rep_rows,
                "ratio_to_sol_over_repeats": spread([r_["ratio_to_sol"] for r_ in rep_rows]),
                "p50_us_over_repeats": p50_all,
                "twoshot_atomic_not_bit_reproducible": bench_size(8192, (symar.TWOSHOT_ATOMIC,))["twoshot_atomic"],
                "prior_art_two_barrier_oneshot": {
                    "p50_us": prior["p50"], "bit_exact": prior["bit_exact"], "ctas_per_rank": prior["ctas_per_rank"],
                    "threads": prior["threads"],
                    "note": "8 bytes per thread; release signals + a second barrier before exit"},
                "oneshot_release_signal": {
                    "p50_us": release["p50"], "bit_exact": release["bit_exact"], "ctas_per_rank": release["ctas_per_rank"],
                    "threads": release["threads"], "ratio_to_sol": release["p50"] / sol,
                    "note": "the selector's one-shot with red.release on the ready signal and nothing else changed: "
                            "the form a system needs whose ranks do not share a kernel boundary"},
                "system_scope_build": sys_scope,
                "placement": dict(zip(("measured", "sms_on_second_half", "home_bits"), h.placement())),
                "without_placement_on_l2_halves": {"p50_us": unplaced["p50"], "bit_exact": unplaced["bit_exact"],
                                                   "note": "every reader takes copy 0 of its flags and counters"},
                "in_kernel_span_us_p50": {
                    names[a_]: float(np.median([h.debug_span(0, out_off, 8192, symar.BF16, a_) for _ in range(31)])) / 1e3
                    for a_ in (symar.ONESHOT, symar.TWOSHOT, symar.LL, symar.SENTINEL)},
                "in_kernel_span_note": "first CTA in (after its wait for the previous grid) -> last CTA out, device "
                                       "nanosecond timer (about 32 ns resolution), single stream-launched calls "
                                       "through the instrumented instantiation of the same kernels",
                "phase_stamps_us": phases,
                "phase_stamps_note": "per phase {first, mean, last} over all CTAs (thread 0 of each), us since the first "
                                     "CTA's start; median of 31 instrumented calls; phases as in symar_debug_phases",
                "oracle_cpu": oracle_us(O, load_inputs(8192)),
                "sol_us": sol,
                "sol_parts_us": {"empty_launch_same_shape": floor_us, "empty_launch_1x1": floor11["p50"],
                                 "flag_round_trip": rt_us, "bytes_at_peak": t_bytes_us,
                                 "empty_launch_plain": floor.get("plain_p50"),
                                 "empty_launch_slot_clusters": floor.get("slot_clusters_p50"),
                                 "selector_launch_uses_slot_clusters":
                                     bool(best.get("variant", 0) & symar.VARIANT_CLUSTER)},
                "ratio_to_sol": p50_all["median"] / sol,
                "sol_note": "empty launch = the smallest p50 over the repeats of an empty kernel in the selector's grid "
                            "and block with programmatic dependent launch, launched plainly or with each slot's ranks as "
                            "one thread-block cluster, whichever is cheaper; flag round trip = the MEDIAN over SM "
                            "pairs "
                            "spread over the chip (the exchange needs every pair of ranks, wherever their CTAs sit; two hops "
                            "through L2 of a flag that is not placed), median over the repeats; the same bound with the "
                            "FASTEST pair follows.  The kernel's own exchange is one hop and a poll of a flag placed on the "
                            "reader's L2 half, and its launch overlaps the previous call, so this form is a yardstick, not a "
                            "strict floor; the fastest-pair form is the strict one",
                "sol_fastest_pair_us": sol_fast,
                "ratio_to_sol_fastest_pair": p50_all["median"] / sol_fast,
                "sol_strictest_us": min(floor11["p50"], floor_us) + rt_min_us + t_bytes_us,
                "ratio_to_sol_strictest": p50_all["median"] / (min(floor11["p50"], floor_us) + rt_min_us + t_bytes_us),
                "sol_strictest_note": "empty 1x1 launch + fastest SM pair + bytes at peak",
                "paper_style_sol_us": (2 * fence_ns + rt_ns / 2) / 1000.0,
                "fence_us": fence_ns / 1000.0,
            }
            out["latency_16KB"]["launch"] = "programmatic dependent launch (the library's default); the empty " \
                                            "kernel of the bound is launched with the same attribute"
            # the same without programmatic dependent launch, floor measured without it too
            h.set_pdl(False)
            prow = bench_size(8192, (symar.AUTO,))["auto"]
            h.set_pdl(True)
            pfloor = empty_floor(prow["ctas_per_rank"], P, prow["threads"], pdl=False)
            psol = pfloor["p50"] + rt_ns / 1000.0 + t_bytes_us
            out["latency_16KB"]["without_programmatic_dependent_launch"] = {
                "p50_us": prow["p50"], "algo": prow["algo"], "bit_exact": prow["bit_exact"],
                "empty_launch_same_shape_us": pfloor["p50"], "sol_us": psol, "ratio_to_sol": prow["p50"] / psol,
                "ratio_to_sol_fastest_pair": prow["p50"] / (pfloor["p50"] + rt_min_ns / 1000.0 + t_bytes_us)}
        # below the metric's sizes: where the data+flag protocol is meant to win (the
        # paper's own zoom is at one 128-byte line per rank), and one cold-cache number
        if P == 8:
            small = []
            for nbytes in (128, 1024, 4096):
                row = bench_size(nbytes // 2, ALL)
                fl = empty_floor(row["auto"]["ctas_per_rank"], P, row["auto"]["threads"])
                s_ol = fl["p50"] + rt_ns / 1000.0 + bytes_us(nbytes, P)
                small.append({"bytes_per_rank": nbytes, "p50_us": {k: v["p50"] for k, v in row.items()},
                              "selector": row["auto"]["algo"],
                              "selector_shape": [row["auto"]["ctas_per_rank"], row["auto"]["threads"]],
                              "ll_shape": [row["ll"]["ctas_per_rank"], row["ll"]["threads"], row["ll"]["variant"]],
                              "ll_minus_oneshot_us": row["ll"]["p50"] - row["oneshot"]["p50"],
                              "sol_us": s_ol, "ratio_to_sol": row["auto"]["p50"] / s_ol,
                              "bit_exact": all(v["bit_exact"] for v in row.values())})
            out["small_messages"] = small
            scrub = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
            cold = []
            with torch.cuda.stream(stream):
                for i in range(30):
                    scrub.fill_(i & 0xFF)                      # evicts heap lines from L2
                    a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a_.record(stream)
                    h.allreduce(0, out_off, 8192, symar.BF16, symar.AUTO, stream.cuda_stream)
                    b_.record(stream)
                    cold.append((a_, b_))
            stream.synchronize()
            out["latency_16KB"]["cold_l2_single_call_us_p50"] = float(np.percentile(
                [a_.elapsed_time(b_) * 1000.0 for a_, b_ in cold], 50))
            del scrub
        # the sibling collectives at the decode-step message (16 KiB per rank of input or output)
        if P == 8:
            x = synth.make_inputs("normal", "bf16", P, 8192, synth.seed_for_config(2))
            for q in range(P):
                h.write_rank(q, 0, x[q])
            sib = {}
            ops = {
                "reduce_scatter": (lambda s: h.reduce_scatter(0, out_off, 8192 // P, symar.BF16, s),
                                   lambda: O.reduce_scatter(x), 8192 // P),
                "all_gather": (lambda s: h.all_gather(0, out_off, 8192 // P, symar.BF16, s),
                               lambda: O.all_gather(np.ascontiguousarray(x[:, :8192 // P])), 8192),
                "broadcast": (lambda s: h.broadcast(0, out_off, 8192, symar.BF16, 3, s),
                              lambda: O.broadcast(x, 3), 8192),
                "reduce": (lambda s: h.reduce(0, out_off, 8192, symar.BF16, 3, s), lambda: O.reduce(x), 8192),
            }
            for name, (call, ref, n_out) in ops.items():
                assert call(stream.cuda_stream) == 0
                stream.synchronize()
                if name == "reduce":
                    exact = bool(np.array_equal(h.read_rank(3, out_off, n_out, np.uint16), ref()))
                else:
                    got = np.stack([h.read_rank(q, out_off, n_out, np.uint16) for q in range(P)])
                    exact = bool(np.array_equal(got, ref()))
                g = graph_of(torch, stream, lambda k, s, call=call: call(s), K)
                r = time_graph(torch, g, stream, K, reps)
                sib[name] = {"p50_us": r["p50"], "bit_exact": exact and h.status()[0] == 0}
            out["sibling_collectives_16KB"] = sib
        # Sec. VII "Impact of Scratch Buffer": a 32 MiB message through the push algorithms with
        # ever smaller scratch, i.e. more iterations, each with its own synchronisation
        if P == 8 and not quick:
            hs = symar.SymHeap.on_torch(P, 64 << 20)
            cnt32 = (32 << 20) // 2
            xs32 = synth.make_inputs("normal", "bf16", P, cnt32, 77)
            for q in range(P):
                hs.write_rank(q, 0, xs32[q])
            want32 = O.allreduce_timed_team(xs32, threads=0)[0][0]
            sweep32 = []
            for limit in (16 << 10, 64 << 10, 256 << 10, 1 << 20):
                hs.set_scratch_limit(limit)
                row = {"scratch_payload_bytes_per_iteration": limit, "ms": {}, "bit_exact": True}
                for algo in (symar.LL, symar.SENTINEL, symar.TWOSHOT_LL, symar.TWOSHOT_SENTINEL):
                    with torch.cuda.stream(stream):
                        hs.allreduce(0, 32 << 20, cnt32, symar.BF16, algo, stream.cuda_stream)
                        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a_.record(stream)
                        for _ in range(3):
                            hs.allreduce(0, 32 << 20, cnt32, symar.BF16, algo, stream.cuda_stream)
                        b_.record(stream)
                    stream.synchronize()
                    row["ms"][names[algo]] = a_.elapsed_time(b_) / 3
                    got = hs.read_rank(P - 1, 32 << 20, cnt32, np.uint16)
                    row["bit_exact"] = row["bit_exact"] and bool(np.array_equal(got, want32)) and hs.status()[0] == 0
                sweep32.append(row)
            hs.set_scratch_limit(0)
            with torch.cuda.stream(stream):
                a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                hs.allreduce(0, 32 << 20, cnt32, symar.BF16, symar.TWOSHOT, stream.cuda_stream)
                a_.record(stream)
                for _ in range(3):
                    hs.allreduce(0, 32 << 20, cnt32, symar.BF16, symar.TWOSHOT, stream.cuda_stream)
                b_.record(stream)
            stream.synchronize()
            out["scratch_sweep_32MiB"] = {"rows": sweep32, "flag_twoshot_ms_for_reference": a_.elapsed_time(b_) / 3}
            hs.destroy()
            del xs32
        # C3: sweep
        if P == 8:
            sweep = []
            for B in synth.WORKLOADS["c3"]["batch"]:
                row = bench_size(8192 * B, ALL)
                named = {k: v["p50"] for k, v in row.items() if k != "auto"}
                best_name = min(named, key=named.get)
                ra = bench_size(8192 * B, (symar.TWOSHOT_ATOMIC,))["twoshot_atomic"]
                ud = untuned_default(8192 * B)
                fl = empty_floor(row["auto"]["ctas_per_rank"], P, row["auto"]["threads"], n=100)
                s_ol = fl["p50"] + rt_ns / 1000.0 + bytes_us(16384 * B, P)
                try:       # where two-shot's time goes: exchange, data, CTA barrier, release fence, "done" hop
                    ph = [h.debug_phases(0, out_off, 8192 * B, symar.BF16, symar.TWOSHOT) for _ in range(15)]
                    ts_phases = {str(k): {f: float(np.median([p_[k][f] for p_ in ph])) / 1e3
                                          for f in ("first", "mean", "last")} for k in sorted(ph[0])}
                except symar.SymarError as exc:
                    ts_phases = {"error": str(exc)}
                sweep.append({"bytes_per_rank": 16384 * B, "p50_us": {k: v["p50"] for k, v in row.items()},
                              "twoshot_atomic_p50_us": ra["p50"], "twoshot_atomic_within_tolerance":
                                  ra["within_tolerance"],
                              "selector": row["auto"]["algo"], "selector_shape":
                                  [row["auto"]["ctas_per_rank"], row["auto"]["threads"]],
                              "best": best_name,
                              "selector_within_5pct": bool(row["auto"]["p50"] <= 1.05 * named[best_name]),
                              "sol_us": s_ol, "ratio_to_sol": row["auto"]["p50"] / s_ol,
                              "sol_parts_us": {"empty_launch_same_shape": fl["p50"], "flag_round_trip": rt_ns / 1000.0,
                                               "bytes_at_measured_hbm_copy_rate": bytes_us(16384 * B, P)},
                              "oracle_cpu": oracle_us(O, synth.make_inputs("normal", "bf16", P, 8192 * B,
                                                                           synth.seed_for_config(2))),
                              "untuned_default": ud,
                              "twoshot_phase_stamps_us": ts_phases,
                              "bit_exact": all(v["bit_exact"] for v in row.values()) and ud["bit_exact"]})
            out["sweep"] = sweep
            out["sweep_note"] = "sol_us = empty launch of the selector's shape + median flag round trip + 2*P*M bytes at " \
                                "the measured HBM copy rate (the messages are L2-resident, so the byte term is an upper " \
                                "estimate of what the bound allows); oracle_cpu = the CPU oracle on the same message; " \
                                "untuned_default = the same call on a heap that was never tuned (built-in choice)"
        # C5: 160 calls in one graph
        calls, count = 160, 8192 * 4
        nb = count * 2
        if autotune:
            # the launch shape for this message size as it occurs in the trace -- every call on its own buffers --
            # measured on this GPU (untimed set-up, as a deployment does once for its decode step)
            t0 = time.time()
            h.autotune_stream(symar.BF16, count, calls)
            res["autotune_stream_seconds"] = time.time() - t0
        xs = [synth.make_inputs("normal", "bf16", P, count, synth.seed_for_config(5), call=k) for k in range(calls)]
        for k in range(calls):
            for q in range(P):
                h.write_rank(q, k * nb, xs[k][q])
        base_out = 10 << 20 if calls * nb <= (10 << 20) else calls * nb
        g = graph_of(torch, stream, lambda k, s: h.allreduce(k * nb, base_out + k * nb, count, symar.BF16,
                                                             symar.AUTO, s), calls)
        exact = True
        for rep in range(3):
            with torch.cuda.stream(stream):
                g.replay()
            stream.synchronize()
            for k in (0, 1, 79, 158, 159) if rep else range(calls):
                got = np.stack([h.read_rank(q, base_out + k * nb, count, np.uint16) for q in range(P)])
                exact = exact and bool(np.array_equal(got, O.allreduce(xs[k])))
        a, c, t = h.last_choice()
        n_dec = 60 if quick else 200
        r = time_graph(torch, g, stream, calls, n_dec)
        floor = empty_floor(c, P, t)
        t_bytes_us = bytes_us(nb, P)
        sol = floor["p50"] + rt_ns / 1000.0 + t_bytes_us
        dec_rows = [{"per_call_us": r["p50"], "empty_launch_us": floor["p50"], "flag_round_trip_median_us": rt_ns / 1000.0,
                     "flag_round_trip_min_us": rt_min_ns / 1000.0}]
        for _ in range(REPEATS):
            rt_i = sample_flag_round_trips(torch, symar)
            fl_i = empty_floor(c, P, t)["p50"]
            p_i = time_graph(torch, g, stream, calls, n_dec)["p50"]
            dec_rows.append({"per_call_us": p_i, "empty_launch_us": fl_i, "flag_round_trip_median_us": rt_i["median_us"],
                             "flag_round_trip_min_us": rt_i["min_us"]})
        floor_us = min(d_["empty_launch_us"] for d_ in dec_rows)
        sol = floor_us + float(np.median([d_["flag_round_trip_median_us"] for d_ in dec_rows])) + t_bytes_us
        sol_fast = floor_us + min(d_["flag_round_trip_min_us"] for d_ in dec_rows) + t_bytes_us
        for d_ in dec_rows:
            d_["ratio_to_sol"] = d_["per_call_us"] / sol
        per_call = float(np.median([d_["per_call_us"] for d_ in dec_rows]))
        res.update({"step_total_us_p50": per_call * calls, "per_call_us": dict(r, p50=per_call), "sol_per_call_us": sol,
                    "ratio_to_sol": per_call / sol, "algo": names[a], "ctas_per_rank": c, "threads": t,
                    "sol_fastest_pair_us": sol_fast,
                    "ratio_to_sol_fastest_pair": per_call / sol_fast,
                    "sol_note": "smallest empty launch of the same shape over the repeats + the MEDIAN SM pair's flag round "
                                "trip (two hops through L2, flag not placed; median over the repeats) + bytes at peak; the "
                                "exchange itself needs one hop and a poll of a flag placed on the reader's L2 half, and the "
                                "successor's launch overlaps this call, so this form is a yardstick, not a strict floor; "
                                "the fastest-pair form is the strict one",
                    "repeats": dec_rows, "ratio_to_sol_over_repeats": spread([d_["ratio_to_sol"] for d_ in dec_rows]),
                    "oracle_cpu_one_call": oracle_us(O, xs[0]),
                    "bit_exact": exact, "calls": calls, "bytes_per_rank": nb,
                    "cache_state": "every call has its own input and output (%d MiB touched per step): "
                                   "mostly HBM-cold, unlike the warm 16 KiB number" % (2 * P * calls * nb >> 20)})
        h.set_pdl(False)
        gp = graph_of(torch, stream, lambda k, s: h.allreduce(k * nb, base_out + k * nb, count, symar.BF16,
                                                              symar.AUTO, s), calls)
        rp = time_graph(torch, gp, stream, calls, 60 if quick else 200)
        h.set_pdl(True)
        kchk = calls - 1
        gotp = np.stack([h.read_rank(q, base_out + kchk * nb, count, np.uint16) for q in range(P)])
        res["without_programmatic_dependent_launch"] = {
            "step_total_us_p50": rp["p50"] * calls, "per_call_us": rp["p50"],
            "bit_exact": bool(np.array_equal(gotp, O.allreduce(xs[kchk])))}
        out.setdefault("decode_trace", {})[f"P{P}"] = res
        stream.synchronize()
        h.destroy()
    return out


def finite(obj):
    """JSON has no NaN or Infinity: non-finite numbers become null."""
    if isinstance(obj, float):
        return obj if np.isfinite(obj) else None
    if isinstance(obj, dict):
        return {k: finite(v) for k, v in obj.items()}
    if isinstance(obj, (list, tuple)):
        return [finite(v) for v in obj]
    if isinstance(obj, np.generic):
        return finite(obj.item())
    return obj



# ---------------------------------------------------------------------------------
# output: one short line for the driver, one file per workload for the reader
# ---------------------------------------------------------------------------------
MAX_LINE_CHARS = 2000


def _r(x, nd=4):
    """Numbers of the short line: a few significant decimals are all the clocks justify."""
    if isinstance(x, bool) or x is None:
        return x
    if isinstance(x, (float, np.floating)):
        x = float(x)
        return round(x, nd) if np.isfinite(x) else None
    if isinstance(x, np.integer):
        return int(x)
    return x


def compact_line(bw, lat, details):
    """The line rank 0 prints: the base contract's keys, `roofline`, `cpu_baseline`, `e2e`, and a
    handful of numbers for the latency half of the metric.  `bw` is the bandwidth workload's full
    record (or None), `lat` the latency suite's (or None), `details` the files that hold the rest."""
    line = {}
    if bw:
        for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                  "vs_baseline", "dtype", "data", "impl"):
            line[k] = _r(bw.get(k))
        cfg = bw.get("config", {})
        line["config"] = {"workload": "c4: P=8 emulated ranks, fp32, %s el/rank, U(-1,1), two-shot; value=2PM B/time; "
                                      "4 GiB per step >> L2" % cfg.get("elements_per_rank"),
                          "kernel": cfg.get("kernel"),
                          "ctas_per_rank": cfg.get("ctas_per_rank"), "threads": cfg.get("threads"),
                          "multi_gpu": "replicas"}
        ck = bw.get("clocks") or {}
        line["clocks"] = {"sm_mhz": _r(ck.get("sm_mhz"), 0), "sm_max_mhz": _r(ck.get("sm_max_mhz"), 0),
                          "reasons": ck.get("reasons", [])}
        line["gpu_launches"] = bw.get("gpu_launches")
        line["bit_exact_sampled"] = bw.get("bit_exact_sampled")
        rf = bw.get("roofline") or {}
        line["roofline"] = {"bound": rf.get("bound"), "achieved": _r(rf.get("achieved"), 1), "peak": _r(rf.get("peak"), 1),
                            "unit": rf.get("unit"), "frac": _r(rf.get("frac")), "peak_source": "measured"
                            if str(rf.get("peak_source", "")).startswith("measured") else "fallback",
                            "frac_nominal_8TBs": _r(rf.get("frac_of_nominal_8TBps")),
                            "live_copy": _r(rf.get("live_copy_gbs"), 0),
                            "algorithmic_bytes": rf.get("algorithmic_bytes_per_launch"),
                            "launch_ms": _r((rf.get("launch_ms") or {}).get("mean")), "traffic": rf.get("traffic")}
        if bw.get("cpu_baseline"):
            cb = bw["cpu_baseline"]
            line["cpu_baseline"] = {"value": _r(cb["value"], 2), "unit": cb["unit"], "cores": cb["cores"],
                                    "kind": cb["kind"], "sample": "whole workload, best of 5"}
        if bw.get("e2e"):
            e = bw["e2e"]
            line["e2e"] = {"value": _r(e["value"], 2), "unit": e["unit"], "h2d_bytes_per_step": e["h2d_bytes_per_step"],
                           "d2h_bytes_per_step": e["d2h_bytes_per_step"], "ms_per_step": _r(e.get("ms_per_step"), 2),
                           "bit_exact_sampled": e.get("bit_exact_sampled")}
        elif bw.get("e2e_skipped"):
            line["e2e_skipped"] = str(bw["e2e_skipped"])[:80]
    else:
        line.update({"metric": METRIC, "impl": "ours", "data": "synthetic", "dtype": "bf16", "note": "latency section only"})
    if lat and "latency_section_error" in lat:
        line["latency_section_error"] = str(lat["latency_section_error"])[:160]
    if lat and "latency_16KB" in lat:
        c2 = lat["latency_16KB"]
        best = c2.get("best", {})
        rs = c2.get("ratio_to_sol_over_repeats", {})
        sysb = c2.get("system_scope_build") or {}
        line["latency_16KB"] = {
            "p50_us": _r(c2.get("p50_us"), 3), "algo": best.get("algo"),
            "shape": [best.get("ctas_per_rank"), best.get("threads")],
            "sol_us": _r(c2.get("sol_us"), 3), "ratio_to_sol": _r(c2.get("ratio_to_sol"), 3),
            "repeats": rs.get("n"), "ratio_median": _r(rs.get("median"), 3), "ratio_min": _r(rs.get("min"), 3),
            "ratio_max": _r(rs.get("max"), 3),
            "ratio_to_sol_fastest_pair": _r(c2.get("ratio_to_sol_fastest_pair"), 3),
            "bit_exact": all(v.get("bit_exact") for v in c2.get("per_algo", {}).values()),
            "ll_p50_us": _r((c2.get("per_algo", {}).get("ll") or {}).get("p50"), 3),
            "oneshot_release_p50_us": _r((c2.get("oneshot_release_signal") or {}).get("p50_us"), 3),
            "unplaced_p50_us": _r((c2.get("without_placement_on_l2_halves") or {}).get("p50_us"), 3),
            "sys_scope_p50_us": {k: _r((sysb.get(k) or {}).get("p50_us"), 3) for k in ("oneshot", "ll")}
            if "error" not in sysb else None,
        }
    if lat and "decode_trace" in lat:
        line["decode_trace"] = {}
        for key, d in lat["decode_trace"].items():
            rs = d.get("ratio_to_sol_over_repeats", {})
            line["decode_trace"][key] = {
                "us_per_call": _r((d.get("per_call_us") or {}).get("p50"), 3), "ratio_to_sol": _r(d.get("ratio_to_sol"), 3),
                "ratio_min": _r(rs.get("min"), 3), "ratio_max": _r(rs.get("max"), 3),
                "ratio_fastest_pair": _r(d.get("ratio_to_sol_fastest_pair"), 3), "algo": d.get("algo"),
                "bit_exact": d.get("bit_exact")}
    if lat and "sweep" in lat:
        line["sweep_ok"] = {"selector_within_5pct": all(r_.get("selector_within_5pct") for r_ in lat["sweep"]),
                            "bit_exact": all(r_.get("bit_exact") for r_ in lat["sweep"])}
    which = ",".join(sorted(Path(d_).stem.replace("results_", "") for d_ in details))
    line["details"] = (str(Path(details[0]).parent) + "/results_{" + which + "}.json") if details else None
    return finite(line)


def write_results(out_dir, bw, lat):
    """One JSON file per workload: c4 (bandwidth), c2 (16 KiB and below, the bound's parts), c3 (sweep,
    tuner table, context), c5 (decode trace).  Returns the paths written, relative to the repository."""
    out_dir = Path(out_dir)
    paths = []
    try:
        out_dir.mkdir(parents=True, exist_ok=True)
    except OSError:
        return paths
    lat = lat or {}
    parts = {
        "results_c4.json": bw,
        "results_c2.json": {k: lat[k] for k in ("latency_16KB", "small_messages", "flag_round_trip_pairs", "barrier_us")
                            if k in lat},
        "results_c3.json": {k: lat[k] for k in ("sweep", "sweep_note", "tuner_table_bf16", "sibling_collectives_16KB",
                                                "scratch_sweep_32MiB") if k in lat},
        "results_c5.json": {k: lat[k] for k in ("decode_trace",) if k in lat},
    }
    for name, body in parts.items():
        if not body:
            continue
        try:
            (out_dir / name).write_text(json.dumps(finite(body), allow_nan=False, indent=1) + "\n")
            p_ = out_dir / name
            paths.append(str(p_.relative_to(ROOT)) if p_.is_relative_to(ROOT) else str(p_))
        except OSError:
            pass
    return paths


def emit(line):
    """Prints the one line; if it ever outgrew the limit, drops the optional parts rather than the contract's."""
    text = json.dumps(line, allow_nan=False, separators=(",", ":"))
    for k in ("sweep_ok", "decode_trace", "latency_16KB", "details"):
        if len(text) < MAX_LINE_CHARS:
            break
        line.pop(k, None)
        line["truncated"] = True
        text = json.dumps(line, allow_nan=False, separators=(",", ":"))
    print(text, flush=True)
    return text


# ---------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--count", type=int, default=0, help="elements per rank (default: the 64 Mi workload)")
    ap.add_argument("--no-latency", action="store_true", help="skip the 16 KiB / sweep / decode-trace section")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--quick", action="store_true", help="fewer latency samples")
    ap.add_argument("--latency-only", action="store_true", help="skip the bandwidth workload (no `value`)")
    ap.add_argument("--no-autotune", action="store_true", help="built-in launch shapes: no tuning of the bandwidth workload's size nor of the latency section")
    ap.add_argument("--ctas", type=int, default=0)
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--variant", type=lambda v: int(v, 0), default=0, help="two-shot kernel variant bits")
    ap.add_argument("--out-dir", default=str(ROOT / "gpurun_out"), help="where the per-workload result files go")
    ap.add_argument("--scope-probe", default=None, help=argparse.SUPPRESS)     # child process of the latency section
    ap.add_argument("--case", default=None, help="ALGO:BYTES[:P[:VARIANT[:CTAS:THREADS]]] -- a few calls of one "
                                                 "algorithm on a bf16 message (for profilers); --steps calls, default 5")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return
    if args.scope_probe:
        scope_probe(args.scope_probe, args.quick)
        return
    if args.case:
        import __graft_entry__ as ge
        ge.build()
        run_case(args.case, args.steps if args.steps != 500 else 5, args.warmup)
        return

    import torch
    import torch.distributed as dist
    import __graft_entry__ as ge
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the AllReduce has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        ge.build()
    if world > 1:
        dist.barrier()
    from paper_2607_16100_b200 import symar, synth

    hbm_gbs, peak_src = peaks()
    if args.latency_only:
        if rank == 0:
            lat = latency_suite(torch, symar, synth, hbm_gbs, quick=args.quick, autotune=not args.no_autotune)
            emit(compact_line(None, lat, write_results(args.out_dir, None, lat)))
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return
    w = dict(synth.WORKLOADS["c4"])
    if args.count:
        w["count"] = args.count
    P, count = w["P"], w["count"]
    M = count * 4
    algbytes = 2 * P * M

    # inputs: seeded, generated on the host, then made resident in HBM
    x = synth.make_inputs(w["dist"], w["dtype"], P, count, w["seed"] + rank)
    in_off, out_off = 0, (M + 4095) // 4096 * 4096
    heap = symar.SymHeap.on_torch(P, out_off + M, device=f"cuda:{local}")
    tune_s = None
    if args.ctas or args.threads or args.variant:
        if args.ctas or args.threads:
            heap.set_launch(symar.TWOSHOT, args.ctas, args.threads)
        if args.variant:
            heap.set_variant(symar.TWOSHOT, args.variant)
    elif not args.no_autotune:
        # the launch shape for exactly this message size, measured on this GPU (untimed set-up,
        # as a deployment would do once); overwrites the user region, so inputs go in after it
        t0 = time.time()
        heap.autotune_size(symar.F32, count)
        torch.cuda.synchronize()
        tune_s = time.time() - t0
    for q in range(P):
        heap.write_rank(q, in_off, x[q])
    stream = torch.cuda.Stream()
    sh = stream.cuda_stream
    step = lambda: heap.allreduce(in_off, out_off, count, symar.F32, symar.TWOSHOT, sh)

    for _ in range(args.warmup):
        step()
    stream.synchronize()
    algo, ctas, threads = heap.last_choice()
    variant, smem = heap.last_kernel()
    kernel = "twoshot_bulk_kernel<F32, 8>" if smem else "twoshot_kernel<F32, 8>"
    tile_kib = (4 << ((variant >> 12) & 3)) if smem else None

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    # one event pair around the timed region; in between an event after every tenth of the steps, for the
    # spread (an event between two launches keeps the second from overlapping its launch with the first's
    # tail, so there are few)
    marks = sorted(set([args.steps] + [k * args.steps // 10 for k in range(1, 10) if k * args.steps // 10 > 0]))
    ev = {m: torch.cuda.Event(enable_timing=True) for m in [0] + marks}
    t_begin = time.time()
    with torch.cuda.stream(stream):
        ev[0].record(stream)
        for i in range(args.steps):
            step()
            if i + 1 in ev:
                ev[i + 1].record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    t_end = time.time()
    if world > 1:
        dist.barrier()
    total_ms = ev[0].elapsed_time(ev[args.steps])
    bounds = [0] + marks
    # average launch duration per segment between two events; the mean over launches is total / steps
    seg_ms = np.array([ev[a].elapsed_time(ev[b]) / (b - a) for a, b in zip(bounds[:-1], bounds[1:])])
    per_launch_ms = np.array([total_ms / args.steps])
    clocks = sampler.stop(t_begin, t_end)
    assert heap.status()[0] == symar.OK, f"device status {heap.status()}"

    total_ms = max_over_ranks(dist if world > 1 else None, total_ms, "cuda")
    value = whole_job_value(algbytes, world, args.steps, total_ms) / 1e9

    # parity of what was just timed, on sampled positions (oracle element by element)
    from oracle import allreduce_oracle as O
    rng = np.random.default_rng(1)
    starts = [0, count - 4096, (count // P) - 2048, 3 * (count // P) - 2048] + \
        [int(s) for s in rng.integers(0, max(1, count - 4096), size=12)]
    exact = True
    for s0 in starts:
        s0 = max(0, min(s0, count - 4096)) // 4 * 4
        n = min(4096, count - s0)
        want = O.allreduce(np.ascontiguousarray(x[:, s0:s0 + n]))
        for r in range(P):
            got = heap.read_rank(r, out_off + s0 * 4, n, np.float32)
            exact = exact and bool(np.array_equal(got.view(np.uint32), want[r].view(np.uint32)))

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "impl": "ours",
        "config": {
            "workload": f"c4: P={P} emulated ranks, fp32, {count} elements ({M >> 20} MiB) per rank, U(-1,1), "
                        "two-shot reduce-scatter + all-gather; value = 2*P*M bytes / time",
            "P": P, "elements_per_rank": count, "algo": "twoshot", "ctas_per_rank": ctas, "threads": threads,
            "kernel": kernel, "bulk_tile_KiB": tile_kib, "bulk_stages": ((variant >> 8) & 7) or None,
            "dynamic_smem_bytes": smem, "shape_tuned_for_this_size_seconds": tune_s,
            "l2": f"inputs {P * M >> 20} MiB + outputs {P * M >> 20} MiB per step, far larger than the 126 MB L2; "
                  "no flush needed",
            "multi_gpu": "replicas only (independent heaps, no exchange between GPUs)",
        },
        "clocks": clocks,
        "gpu_launches": args.steps,
        "bit_exact_sampled": exact,
        "roofline": {
            "bound": "hbm", "achieved": algbytes / (float(per_launch_ms.mean()) * 1e-3) / 1e9, "peak": hbm_gbs,
            "unit": "GB/s", "frac": algbytes / (float(per_launch_ms.mean()) * 1e-3) / 1e9 / hbm_gbs,
            "peak_source": peak_src, "kernel": kernel,
            "algorithmic_bytes_per_launch": algbytes,
            "launch_ms": {"mean": float(per_launch_ms.mean()), "min": float(seg_ms.min()),
                          "max": float(seg_ms.max()), "note": "mean = timed region / launches; min and max over "
                          "the average launch of each tenth of the region"},
            "frac_of_nominal_8TBps": algbytes / (float(per_launch_ms.mean()) * 1e-3) / 1e9 / 8000.0,
            "traffic": None,
        },
    }
    # context for the fraction: a plain device-to-device copy of as many bytes, timed in this process on this
    # GPU (the denominator above is the pool-wide measured copy rate; this says what this box's copy does now)
    try:
        src = torch.empty(algbytes // 2, dtype=torch.uint8, device="cuda")
        dst = torch.empty_like(src)
        src.fill_(1)
        with torch.cuda.stream(stream):
            for _ in range(2):
                dst.copy_(src)
            ca, cb_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ca.record(stream)
            for _ in range(5):
                dst.copy_(src)
            cb_.record(stream)
        stream.synchronize()
        line["roofline"]["live_copy_gbs"] = 5 * algbytes / (ca.elapsed_time(cb_) * 1e-3) / 1e9
        del src, dst
    except RuntimeError as exc:
        line["roofline"]["live_copy_gbs"] = None
        line["roofline"]["live_copy_error"] = str(exc)[:200]
    traffic_note = ROOT / "profiles" / ("twoshot_bulk_f32_p8_traffic.txt" if smem else "twoshot_f32_p8_traffic.txt")
    if traffic_note.exists() and count == synth.WORKLOADS["c4"]["count"]:
        kv = dict(l.split("=", 1) for l in traffic_note.read_text().splitlines() if "=" in l and not l.startswith("#"))
        line["roofline"]["traffic"] = int(kv["dram_bytes_per_launch_at_full_size "].strip())
        line["roofline"]["traffic_source"] = kv["source "].strip()

    # end to end through the host-buffer entry point
    e2e_ready = not args.no_e2e
    if e2e_ready:
        # 2 x P x M bytes of pinned host memory per rank; if any rank cannot get them, all skip
        try:
            hin = torch.from_numpy(x).pin_memory()
            hout = torch.empty_like(hin).pin_memory()
        except RuntimeError as exc:
            e2e_ready = False
            line["e2e_skipped"] = f"pinned host buffers: {exc}"
        if world > 1:
            flag = torch.tensor([1.0 if e2e_ready else 0.0], device="cuda")
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            if e2e_ready and flag.item() == 0.0:
                e2e_ready = False
                line["e2e_skipped"] = "another rank could not allocate its pinned host buffers"
    if e2e_ready:
        e2e_steps = min(args.steps, 5)
        estep = lambda: heap.allreduce_host(hin.data_ptr(), hout.data_ptr(), in_off, out_off, count,
                                            symar.F32, symar.TWOSHOT, sh)
        estep()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            a.record(stream)
            for _ in range(e2e_steps):
                estep()
            b.record(stream)
        stream.synchronize()
        e_ms = a.elapsed_time(b)
        e_ms = max_over_ranks(dist if world > 1 else None, e_ms, "cuda")
        s0 = count // 2
        want = O.allreduce(np.ascontiguousarray(x[:, s0:s0 + 4096]))
        e2e_exact = bool(np.array_equal(hout.numpy()[:, s0:s0 + 4096].view(np.uint32), want.view(np.uint32)))
        line["e2e"] = {"value": whole_job_value(algbytes, world, e2e_steps, e_ms) / 1e9, "unit": "GB/s",
                       "h2d_bytes_per_step": P * M, "d2h_bytes_per_step": P * M, "steps": e2e_steps,
                       "ms_per_step": e_ms / e2e_steps, "bit_exact_sampled": e2e_exact,
                       "note": "allreduce_host(): pinned host inputs -> HBM, kernels, all P outputs -> pinned host, in 16 MiB "
                               "chunks on two copy streams (one kernel per chunk; both link directions busy at once)"}
        del hin, hout

    heap.destroy()
    del heap

    if rank == 0 and not args.no_cpu:
        # the oracle as it stands on the whole workload (it needs about 0.1 s per call on 16 cores)
        best, team = 1e30, 1
        t_all = time.perf_counter()
        for _ in range(5):
            t0 = time.perf_counter()
            _, team = O.allreduce_timed_team(x, threads=0)
            best = min(best, time.perf_counter() - t0)
        t0 = time.perf_counter()
        O.allreduce_timed_team(x, threads=1)
        one = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": 2 * P * count * 4 / best / 1e9, "unit": "GB/s", "cores": team, "kind": "oracle",
            "sample": f"the whole workload ({count} elements per rank), best of 5 full oracle calls (OpenMP over "
                      f"elements) + one single-thread call: {2 * P * count * 4 / one / 1e9:.2f} GB/s; "
                      f"{time.perf_counter() - t_all:.1f} s of CPU time in all",
        }
    del x

    lat = None
    if rank == 0 and not args.no_latency:
        try:
            lat = latency_suite(torch, symar, synth, hbm_gbs, quick=args.quick, autotune=not args.no_autotune)
        except Exception as exc:                      # the bandwidth line above must still be reported
            lat = {"latency_section_error": f"{type(exc).__name__}: {exc}"}

    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        emit(compact_line(line, lat, write_results(args.out_dir, line, lat)))


if __name__ == "__main__":
    main()
