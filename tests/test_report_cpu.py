"""The table maker reads what bench.py prints: a made-up line with every kind of
entry (headline, workload list, sweep cells in both split modes, RUN-mask
series, the reference arm) has to come out as the tables it describes."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2609_37062_b200 import report  # noqa: E402

CLOCKS = {"sm_mhz": 1965, "sm_max_mhz": 1965, "reasons": []}


def _entry(workload, us, kv_bytes, **more):
    e = {"workload": workload, "split": "auto", "us_per_step": us, "us_per_step_min": us - 0.1, "steps": 20, "repeats": 30,
         "logical_kv_bytes": kv_bytes, "unique_kv_bytes": kv_bytes, "GB/s": kv_bytes / us / 1e3,
         "pct_of_8tbs": kv_bytes / us / 1e3 / 80.0, "pct_of_measured_hbm": kv_bytes / us / 1e3 / 65.0, "units": 512,
         "chunk_tokens": 256, "max_splits": 1, "copies": 10, "clocks": CLOCKS}
    e.update(more)
    return e


def _line():
    kv = 128 << 20
    return {
        "metric": "decode-attn KV-read GB/s", "value": 5800.0, "unit": "GB/s", "n_gpus": 1, "steps": 20, "warmup": 5,
        "repeats": 100, "ms_per_step": 0.0232, "us_per_step": 23.2, "us_per_step_min": 23.1, "pct_of_8tbs": 72.5,
        "pct_of_measured_hbm": 88.6,
        "config": {"workload": "long_32k", "replan": {"plan_destroy_us_median": 21.0, "plan_destroy_us_p90": 23.0,
                                                       "plan_update_us_median": 12.0, "plan_update_us_p90": 12.5}},
        "roofline": {"kernel_only": {"us_per_launch": 21.8, "frac": 0.94}},
        "gather_probe": {"us_per_step": 25.9, "GB/s": 5180.0},
        "e2e": {"value": 53.0, "ms_per_step": 2.5}, "e2e_resident_kv": {"value": 1400.0, "ms_per_step": 0.095},
        "cpu_baseline": {"value": 4.5, "cores": 16}, "clocks": CLOCKS,
        "configs": [
            _entry("short_chat", 20.0, 96 << 20, cpu_baseline={"cores": 16, "ms_per_step": 17.0, "value": 5.6},
                   replan={"plan_destroy_us_median": 21.5, "plan_destroy_us_p90": 22.5}),
            _entry("shared_prefix", 50.0, 1600 << 20, unique_kv_bytes=140 << 20, shared_prefix_tokens=1536),
            _entry("sweep_8192x64", 300.0, 2 << 30, gather_probe={"GB/s": 7000.0}),
            _entry("sweep_8192x64", 330.0, 2 << 30, split="deterministic"),
            _entry("sweep_1024x256", 150.0, 1 << 30, masked_fraction=0.0, read_kv_bytes=1 << 30),
            _entry("sweep_1024x256", 84.0, 1 << 30, masked_fraction=0.5, read_kv_bytes=1 << 29),
            _entry("sweep_1024x256", 10.0, 1 << 30, masked_fraction=1.0, read_kv_bytes=0),
        ],
    }


def test_tables_from_a_bench_line(tmp_path, capsys):
    path = tmp_path / "line.json"
    ref = {"impl": "reference", "value": 4.4, "ms_per_step": 30.5, "cpu_baseline": {"cores": 16, "sample": "whole batch"}}
    path.write_text("some log line\n" + json.dumps(ref) + "\n" + json.dumps(_line()) + "\n")
    report.main([str(path)])
    out = capsys.readouterr().out
    assert "reference arm (the oracle): 4.40 GB/s, 30.5 ms per step, 16 cores" in out
    assert "### long_32k (1 GPU, 20 steps per region, 100 regions)" in out
    assert "| us per step, median of regions (fastest region) | 23.20 (23.10) |" in out
    assert "| partial kernel alone, us per launch (fraction of measured) | 21.80 (0.940) |" in out
    assert "| in-place refresh (plan_update) us, median / p90 | 12.0 / 12.5 |" in out
    assert "| shared_prefix | auto, shared prefix 1536 | 50.00 (49.90) |" in out
    assert "| | oracle on 16 host cores | 17.0 ms per step | 5.60 |" in out
    # the two split modes of a cell side by side, with their ratio and the probe
    row = next(ln for ln in out.splitlines() if ln.startswith("| 8192 x 64 |"))
    assert "| 2 GiB |" in row and "300.0 (299.9)" in row and "330.0 (329.9)" in row and "| 1.10 | 7000 |" in row
    # the mask series against the straight line between no row and every row masked
    half = next(ln for ln in out.splitlines() if ln.startswith("| 0.5 |"))
    assert "| 80.0 | 1.050 |" in half and "| 537 |" in half


def test_usage_without_arguments():
    try:
        report.main([])
    except SystemExit as e:
        assert "bench.py" in str(e)
    else:
        raise AssertionError("expected the usage text")
