"""The line bench.py prints must stay short: whoever runs the benchmark keeps only the tail of
stdout, and a line that does not fit is a benchmark without a result.  Built here from canned
numbers (no GPU), with every optional part present and every number at full float width."""
import io
import json
import sys
from contextlib import redirect_stdout
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

import bench  # noqa: E402

F = 1234.56789012345678            # a float that prints at full width


def canned_bandwidth_record():
    return {
        "metric": bench.METRIC, "value": 6570.123456789012, "unit": "GB/s", "n_gpus": 1, "steps": 500, "warmup": 5,
        "ms_per_step": 0.6536512345678901, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "impl": "ours",
        "config": {"workload": "w" * 300, "P": 8, "elements_per_rank": 67108864, "algo": "twoshot", "ctas_per_rank": 16,
                   "threads": 512, "kernel": "twoshot_bulk_kernel<F32, 8>", "bulk_tile_KiB": 8, "bulk_stages": 2,
                   "dynamic_smem_bytes": 155776, "shape_tuned_for_this_size_seconds": 2.123456789, "l2": "x" * 200,
                   "multi_gpu": "y" * 100},
        "clocks": {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "samples": 12, "reasons": ["sw_power_cap"]},
        "gpu_launches": 500, "bit_exact_sampled": True,
        "roofline": {"bound": "hbm", "achieved": F * 5, "peak": 6546.2, "unit": "GB/s", "frac": 1.0037123456789,
                     "peak_source": "measured (MEASURED_PEAKS.json hbm_gbs)", "kernel": "twoshot_bulk_kernel<F32, 8>",
                     "algorithmic_bytes_per_launch": 4294967296,
                     "launch_ms": {"mean": 0.65365123456, "min": 0.6501234567, "max": 0.6601234567},
                     "frac_of_nominal_8TBps": 0.82134567891, "live_copy_gbs": 6543.21987654321, "traffic": 3893700198, "traffic_source": "z" * 200},
        "cpu_baseline": {"value": 59.512345678, "unit": "GB/s", "cores": 16, "kind": "oracle", "sample": "s" * 300},
        "e2e": {"value": 90.912345678, "unit": "GB/s", "h2d_bytes_per_step": 2147483648, "d2h_bytes_per_step": 2147483648,
                "steps": 5, "ms_per_step": 47.2123456789, "bit_exact_sampled": True, "note": "n" * 300},
    }


def canned_latency_record():
    algo_row = {"p10": F / 1000, "p50": F / 1000, "p90": F / 1000, "algo": "twoshot_sentinel", "ctas_per_rank": 160,
                "threads": 512, "variant": 0x8100, "bit_exact": True, "stream_launched_p50": F / 1000}
    per_algo = {n: dict(algo_row) for n in ("oneshot", "twoshot", "ll", "sentinel", "twoshot_ll", "twoshot_sentinel",
                                            "auto")}
    spread = {"median": 1.2345678901, "min": 1.1234567891, "max": 1.2987654321, "n": 5}
    rep = {"p50_us": F / 1000, "empty_launch_us": 0.5, "flag_round_trip_median_us": 0.9, "flag_round_trip_min_us": 0.47,
           "sol_us": 1.42, "ratio_to_sol": 1.23456789, "ratio_to_sol_fastest_pair": 1.7}
    dec = {"autotune_seconds": 4.5, "step_total_us_p50": 346.64, "per_call_us": {"p10": 2.1, "p50": 2.16650003567338,
                                                                                 "p90": 2.2},
           "sol_per_call_us": 1.9573064848973445, "ratio_to_sol": 1.1068782801212693, "ratio_to_sol_fastest_pair": 1.6123456789, "algo": "twoshot_sentinel",
           "ctas_per_rank": 64, "threads": 128, "repeats": [dict(rep)] * 5, "ratio_to_sol_over_repeats": dict(spread),
           "bit_exact": True, "calls": 160, "bytes_per_rank": 65536, "cache_state": "c" * 200}
    return {
        "flag_round_trip_pairs": {"min_us": 0.47, "median_us": 0.89, "max_us": 1.03,
                                  "pairs": [{"first_block": i, "partner_block": i + 1, "smids": [i, i + 1],
                                             "round_trip_us": 0.9} for i in range(36)]},
        "barrier_us": {"P8": {"relaxed": 0.48, "release_acquire": 1.14}},
        "latency_16KB": {
            "p50_us": 1.8461234567, "best": dict(algo_row), "per_algo": per_algo, "repeats": [dict(rep)] * 5,
            "ratio_to_sol_over_repeats": dict(spread), "p50_us_over_repeats": dict(spread),
            "oneshot_release_signal": {"p50_us": 2.3123456789, "bit_exact": True},
            "without_placement_on_l2_halves": {"p50_us": 1.9876543219, "bit_exact": True},
            "system_scope_build": {"oneshot": {"p50_us": 2.5123456789, "bit_exact": True},
                                   "ll": {"p50_us": 3.0123456789, "bit_exact": True}},
            "oracle_cpu": {"single_thread_us": 123.456789, "all_cores_us": 45.6789123, "cores": 16},
            "sol_us": 1.4231234567, "ratio_to_sol": 1.2971234567, "sol_fastest_pair_us": 1.0123456789,
            "ratio_to_sol_fastest_pair": 1.8312345678, "phase_stamps_us": {"oneshot": {"0": {"first": 0.0}}},
        },
        "small_messages": [{"bytes_per_rank": 128}],
        "sweep": [{"bytes_per_rank": 16384 << i, "selector_within_5pct": True, "bit_exact": True} for i in range(7)],
        "tuner_table_bf16": {"P8": [{"bytes_per_rank": 1 << i, "us": {"oneshot": 1.0}} for i in range(5, 24)]},
        "decode_trace": {"P8": dict(dec), "P4": dict(dec)},
    }


def test_the_printed_line_is_short_and_carries_what_the_contract_asks_for(tmp_path):
    bw, lat = canned_bandwidth_record(), canned_latency_record()
    details = bench.write_results(tmp_path, bw, lat)
    line = bench.compact_line(bw, lat, ["gpurun_out/results_c2.json", "gpurun_out/results_c3.json",
                                        "gpurun_out/results_c4.json", "gpurun_out/results_c5.json"])
    buf = io.StringIO()
    with redirect_stdout(buf):
        text = bench.emit(line)
    assert len(text) < bench.MAX_LINE_CHARS - 100, len(text)          # with room to spare
    assert "truncated" not in text
    # what a reader of the last 3000 characters of stdout gets
    got = json.loads(("noise\n" * 10 + buf.getvalue())[-3000:].splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "gpu_launches", "roofline", "cpu_baseline", "e2e",
                "latency_16KB", "decode_trace", "details"):
        assert key in got, key
    assert got["value"] > 0 and got["config"]["workload"].startswith("c4")
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in got["roofline"]
    assert got["e2e"]["h2d_bytes_per_step"] == 2147483648
    assert got["cpu_baseline"]["kind"] == "oracle" and got["cpu_baseline"]["cores"] == 16
    l16 = got["latency_16KB"]
    assert l16["ratio_median"] == 1.235 and l16["ratio_max"] == 1.299 and l16["repeats"] == 5
    assert l16["oneshot_release_p50_us"] == 2.312 and l16["sys_scope_p50_us"]["ll"] == 3.012
    assert got["decode_trace"]["P4"]["us_per_call"] == 2.167
    # the details went to one file per workload
    assert sorted(Path(p).name for p in details) == ["results_c2.json", "results_c3.json", "results_c4.json",
                                                     "results_c5.json"]
    c2 = json.loads((tmp_path / "results_c2.json").read_text())
    assert len(c2["flag_round_trip_pairs"]["pairs"]) == 36 and "per_algo" in c2["latency_16KB"]
    assert "sweep" in json.loads((tmp_path / "results_c3.json").read_text())


def test_a_line_that_outgrows_the_limit_loses_its_optional_parts_not_the_contract():
    bw, lat = canned_bandwidth_record(), canned_latency_record()
    line = bench.compact_line(bw, lat, ["d" * 3000 + "/results_c2.json"])
    buf = io.StringIO()
    with redirect_stdout(buf):
        text = bench.emit(line)
    got = json.loads(text)
    assert len(text) < bench.MAX_LINE_CHARS and got["truncated"] is True
    for key in ("metric", "value", "roofline", "cpu_baseline", "e2e"):
        assert key in got


def test_latency_only_and_failed_latency_section_still_give_a_line():
    line = bench.compact_line(None, canned_latency_record(), [])
    assert line["note"] == "latency section only" and "latency_16KB" in line
    line = bench.compact_line(canned_bandwidth_record(), {"latency_section_error": "RuntimeError: " + "e" * 500}, [])
    assert len(json.dumps(line, separators=(",", ":"))) < bench.MAX_LINE_CHARS
    assert "latency_section_error" in line and line["value"] > 0
