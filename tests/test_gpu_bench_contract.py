"""The benchmark driver's JSON line, checked on a short run. Needs a B200."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    """A short run of the default workload (8192^3, three timed steps, reduced extras): one JSON
    line with the metric, the roofline of the dominant kernel, the CPU baseline, the end-to-end
    figure with its copied bytes, the launch count and the clocks seen during the timed region."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "3", "--warmup", "3", "--e2e-steps", "1",
           "--cpu-rows", "64", "--no-sweep", "--probe-ms", "300"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["metric"] == "dgemm_fp64_tflops" and line["unit"] == "TFLOP/s" and line["dtype"] == "f64"
    assert line["n_gpus"] == 1 and line["steps"] == 3 and line["warmup"] == 3 and line["higher_is_better"] is True
    assert line["data"] == "synthetic" and line["vs_baseline"] is None and "workload" in line["config"]
    flop = 2.0 * 8192 ** 3
    assert abs(line["value"] - flop / (line["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * line["value"]
    roof = line["roofline"]
    assert roof["bound"] == "tensor" and roof["unit"] == "TFLOP/s"
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert 0.5 < roof["frac"] <= 1.05          # the kernel is doing the work, and not more than the pipe can (loose: a shared box may run at other clocks)
    assert roof["traffic"] is None or roof["traffic"] > roof["algorithmic_bytes_per_launch"]
    # one GEMM kernel and one reduction kernel per step
    assert line["gpu_launches"] == 2 * line["steps"]
    e2e = line["e2e"]
    assert e2e["unit"] == "TFLOP/s" and 0 < e2e["value"] < line["value"]
    assert e2e["h2d_bytes_per_step"] == 3 * 8192 * 8192 * 8 and e2e["d2h_bytes_per_step"] == 8192 * 8192 * 8
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["cores"] >= 1 and cpu["sample"]
    clocks = line["clocks"]
    assert clocks["sm_max_mhz"] > 0 and clocks["sm_mhz"] > 0 and isinstance(clocks["reasons"], list)
    for bad in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"):
        assert bad not in clocks["reasons"]
