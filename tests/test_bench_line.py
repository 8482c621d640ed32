"""The benchmark's last stdout line is what gets recorded: it must stay a short, complete JSON
object.  CPU checks on the pure assembly functions and on the reference arm; a GPU check on a
real (small) run."""
import argparse
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2608_24070_b200 import inputs as si  # noqa: E402

LIMIT = 2000
REQUIRED = ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
            "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "gpu_launches", "roofline", "cpu_baseline",
            "e2e")
ROOFLINE_KEYS = ("bound", "achieved", "peak", "unit", "frac", "traffic")


def _worst_case_line():
    """Every field at a realistic upper length (seven-digit times, the longest workload key)."""
    args = argparse.Namespace(steps=1000, warmup=100)
    wl = si.WORKLOADS["c4_llama7b_adapter"]
    roof = {"kernel": "sparse_gemm_quad/pair_kernel (fwd, dX)", "bound": "tensor",
            "achieved": 2507.123, "peak": 3386.0, "unit": "TFLOP/s", "frac": 0.7404, "traffic": 507123456,
            "algorithmic_bytes": 398123456,
            "traffic_source": "ncu 16384 tok x1, src 01234567", "peak_source": "2x measured burst cuBLAS",
            "frac_sustained": 0.8906,
            "frac_datasheet": 0.5571, "frac_clock": 0.7312, "frac_kernel_clock": 0.8912, "tflop_per_step": 13.4269,
            "kernel_ms_per_step": 5.3571}
    other = dict(roof, kernel="dense_gemm_pair_kernel (masked dW)")
    clocks = {"sm_mhz": 1417.5, "sm_mhz_min": 1012.5, "sm_max_mhz": 1965.0, "power_w_max": 1002.02, "samples": 1234,
              "window": "x", "reasons": ["hw_slowdown", "hw_thermal_slowdown", "sw_power_cap", "sw_thermal_slowdown"]}
    stage_ms = {op: 12.345 for op in bench.OPS}
    out = bench.headline(args, wl, 16384, 8, 12345.67, 11.6123, 1234.56, 123456, clocks, roof, other, 11.7123, stage_ms,
                         {"sparse": 1172.5, "dense": 1095.5})
    dl = {"dense_ms": 14.4512, "inhouse_dense_ms": 13.9012, "slope_ms": 10.0212, "speedup": 1.443,
          "speedup_vs_inhouse_dense": 1.387}
    e2e = {"value": 431.12, "unit": "TFLOP/s", "ms_per_step": 47.291, "h2d_bytes_per_step": 2560000000,
           "d2h_bytes_per_step": 200000000, "steps": 5, "note": "n" * 300}
    cb = {"value": 0.020512345, "unit": "TFLOP/s", "cores": 128, "kind": "oracle", "seconds": 15.21,
          "sample": "bounded sample: down 11008->4096 b=16384: fwd+dX 1024 token rows, dW 1024 rows",
          "full_workload": False, "extrapolated_step_seconds": 990.1, "extrapolation": "e" * 200}
    bench.attach_extras(out, dl, e2e, cb)
    return out, bench.compact_line(out)


def test_slope_line_is_short_and_complete():
    out, line = _worst_case_line()
    assert len(line) <= LIMIT, len(line)
    assert "\n" not in line
    d = json.loads(line)
    for k in REQUIRED:
        assert k in d, k
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] > 0
    for k in ROOFLINE_KEYS:
        assert k in d["roofline"], k
    assert d["roofline"]["frac"] == pytest.approx(d["roofline"]["achieved"] / d["roofline"]["peak"], abs=2e-4)
    assert set(d["cpu_baseline"]) >= {"value", "unit", "cores", "kind", "sample"}
    assert set(d["e2e"]) >= {"value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"}
    assert "model" not in d["config"] and d["config"]["workload"] == "c4_llama7b_adapter"


def test_an_overlong_line_sheds_detail_and_is_refused_only_when_that_is_not_enough():
    out, line = _worst_case_line()
    out["cpu_baseline"]["sample"] = "whole workload: " + "; ".join(["layer 768->3072 b=8192: fwd+dX 8192 token rows, dW 3072 rows"] * 6)
    shorter = bench.compact_line(out)
    assert len(shorter) <= LIMIT
    d = json.loads(shorter)
    assert d["value"] > 0 and d["roofline"]["frac"] > 0 and d["cpu_baseline"]["value"] > 0 and d["e2e"]["value"] > 0
    assert d["cpu_baseline"]["sample"].endswith("...")
    out["junk"] = "x" * LIMIT
    with pytest.raises(SystemExit):
        bench.compact_line(out)


def test_reference_line_is_short_and_complete(capsys):
    args = argparse.Namespace(workload="c1_single_512", warmup=0, steps=1, gpus=1)
    bench.run_reference(args, rank=0)
    line = capsys.readouterr().out.strip().splitlines()[-1]
    assert len(line) <= LIMIT
    d = json.loads(line)
    assert d["impl"] == "reference" and d["value"] > 0
    assert d["e2e"]["value"] == d["value"] and d["cpu_baseline"]["value"] == d["value"]


def test_recorded_traffic_describes_the_current_kernels():
    """The DRAM traffic in the line comes from an ncu capture; it may only be reported for the
    kernel sources that were captured.  Refresh or clear bench.NCU_TRAFFIC after changing kernels."""
    rec = bench.NCU_TRAFFIC
    if rec["sources"] is None:
        assert rec["sparse_bytes_per_launch"] is None and rec["dense_bytes_per_launch"] is None
        assert bench.recorded_traffic("sparse", "c4_llama7b_adapter", 16384)[0] is None
    else:
        assert rec["sources"] == bench.kernel_sources_sha256()
        t, src = bench.recorded_traffic("sparse", "c4_llama7b_adapter", 16384)
        assert t == round(rec["sparse_bytes_per_launch"] * 16384 / rec["captured_tokens"]) and "ncu" in src


def test_algorithmic_bytes_follow_the_operand_sizes():
    b, d_in, d_out, r = 16384, 4096, 11008, 64
    w = d_in * d_out * 9 // 8
    assert bench.algorithmic_bytes("linear_fwd", b, d_in, d_out, 0) == 2 * b * d_in + w + 2 * b * d_out
    assert bench.algorithmic_bytes("linear_bwd_dx", b, d_in, d_out, r) == \
        2 * b * d_out + w + 2 * b * d_in + 2 * b * r + 2 * r * d_in
    assert bench.algorithmic_bytes("linear_bwd_dw_masked", b, d_in, d_out, r) == 2 * b * (d_in + d_out) + w


@pytest.mark.gpu
def test_a_real_run_ends_in_a_parsable_line(tmp_path):
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    side = tmp_path / "side.json"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "c1_single_512", "--steps", "3",
                          "--warmup", "3", "--side-file", str(side)], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = res.stdout.strip().splitlines()[-1]
    assert len(line) <= LIMIT
    d = json.loads(line)
    for k in REQUIRED:
        assert k in d, k
    assert d["value"] > 0 and d["gpu_launches"] > 0
    assert d["roofline"]["achieved"] > 0 and d["cpu_baseline"]["value"] > 0 and d["e2e"]["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert json.loads(side.read_text())["stages"]
