"""The last stdout line of bench.py is one compact JSON object whatever the size of the per-case
table: the table goes to a file and to earlier "CASE " lines.  Checked on CPU with a table as long
as the real one (49 cases with every optional field)."""
import io
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _fake_case(i):
    return {"config": 6, "layer": "paper_N7168_K18432", "M": 256, "K": 18432, "N": 7168, "path": "gemm_tile_kernel",
            "us": 65.27 + i, "us_min": 64.9, "eff_GBps": 1252.5, "tflops": 1036.39, "bound": "tensor",
            "roofline_frac": 0.6259, "roofline_frac_nominal": 0.46, "split_k": 0, "chosen_split_k": 2,
            "us_by_split_k": {"1": 98.1, "2": 65.2, "4": 70.3, "8": 81.0, "16": 99.9}, "us_split_k_1": 98.1,
            "best_explicit_split_k": 2, "auto_vs_best_explicit": 1.001, "splitk_speedup": 1.5,
            "torch_fp16_matmul_us": 60.1, "speedup_vs_fp16": 0.92}


def _fake_summary():
    return {
        "metric": bench.METRIC, "value": 2237.12, "unit": bench.UNIT, "n_gpus": 1, "steps": 20, "warmup": 5,
        "ms_per_step": 0.052741, "ms_per_step_min": 0.052101, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": bench.WORKLOAD, "group": 128, "accumulate": "f32", "split_k": 0,
                   "l2": "cold: 23 packed weight copies (494 MB) rotated, every call reads HBM",
                   "launch": "one CUDA graph of the 20 steps, replayed 143 times; ms_per_step = median replay",
                   "timed_s": 0.1508, "multi_gpu": "replicas only"},
        "clocks": {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"], "samples": 7},
        "e2e": {"value": 641.2, "unit": bench.UNIT, "h2d_bytes_per_step": 682496, "d2h_bytes_per_step": 253952,
                "ms_per_step": 0.184, "steps": 200, "note": "x" * 90},
        "gpu_launches": 14300,
        "roofline": {"bound": "hbm", "kernel": "gemm_decode_kernel", "launches": "y" * 70, "achieved": 2237.1,
                     "peak": 6537.0, "peak_kind": "of measured", "unit": "GB/s", "frac": 0.3422,
                     "frac_of_nominal_8TBps": 0.2796, "traffic": 23817984, "algorithmic_bytes_per_launch": 23611596,
                     "launch_us": 10.548, "launch_us_by_M": {str(m): 10.0 for m in bench.SWEEP_M},
                     "frac_by_M": {str(m): 0.35 for m in bench.SWEEP_M}, "heaviest_launch": "M=16: gemm_decode_kernel"},
        "roofline_tensor": {"bound": "tensor", "kernel": "gemm_tile_kernel", "case": "M=4096 K=8192 N=8192",
                            "achieved": 1320.1, "peak": 1655.8, "peak_kind": "z" * 70, "unit": "TFLOP/s",
                            "frac": 0.7973, "frac_of_sustained_peak": 0.9412, "frac_of_nominal_2250": 0.5867,
                            "launch_us": 416.3, "traffic": 192325632},
        "config4_block_us_by_M": {"1": 40.7, "16": 56.0, "64": 72.7},
        "cpu_baseline": {"value": 0.08412, "unit": bench.UNIT, "cores": 16, "kind": "oracle", "sample": "s" * 70,
                         "max_elem_err_vs_gpu": 0.00046},
    }


def test_last_line_is_compact_json_and_the_table_goes_elsewhere(tmp_path):
    cases = [_fake_case(i) for i in range(49)]
    out = io.StringIO()
    path = tmp_path / "sub" / "cases.json"
    bench.emit(_fake_summary(), cases, str(path), out)
    lines = out.getvalue().splitlines()
    assert len(lines) == 50 and all(l.startswith("CASE ") for l in lines[:-1])
    last = lines[-1]
    assert len(last.encode()) < 4096
    d = json.loads(last)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "dtype", "config", "clocks", "roofline", "roofline_tensor", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in d
    assert "cases" not in d and d["value"] > 0 and d["config"]["workload"].startswith("config2")
    assert {"frac", "traffic", "achieved", "peak", "bound", "unit"} <= set(d["roofline"])
    assert {"h2d_bytes_per_step", "d2h_bytes_per_step", "value"} <= set(d["e2e"])
    saved = json.load(open(path))
    assert len(saved["cases"]) == 49 and saved["summary"]["value"] == d["value"]
    for l in lines[:-1]:
        json.loads(l[5:])


def test_an_unwritable_cases_file_does_not_break_the_last_line():
    out = io.StringIO()
    bench.emit(_fake_summary(), [_fake_case(0)], "/proc/forbidden/cases.json", out)
    assert json.loads(out.getvalue().splitlines()[-1])["value"] > 0
