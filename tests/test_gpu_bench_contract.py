"""The bench's JSON line carries every key its contract names (run on the small configuration)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "small", "--steps", "3",
           "--warmup", "3", "--no-cpu-baseline", "--no-teacher"]
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks"):
        assert key in line, key
    assert line["steps"] == 3 and line["n_gpus"] == 1 and line["vs_baseline"] is None
    assert line["value"] > 0 and line["ms_per_step"] > 0
    assert "workload" in line["config"] and "model" not in line["config"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in line["roofline"], key
    assert abs(line["roofline"]["frac"] - line["roofline"]["achieved"] / line["roofline"]["peak"]) < 1e-9
    # one denominator whatever the run length (the burst figure), the sustained one beside it
    assert line["roofline"]["frac"] == line["roofline"]["frac_of_burst"]
    assert line["roofline"]["frac_of_sustained"] > line["roofline"]["frac_of_burst"]
    assert line["denoise_pass_all_kernels"]["ms_mean"] >= line["denoise_pass"]["kernel_ms_mean"]
    for key in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert key in line["e2e"], key
    assert line["e2e"]["h2d_bytes_per_step"] > 0 and line["e2e"]["d2h_bytes_per_step"] > 0
    # 4 denoise passes (K rotation + fused kernel) and one commit (2 kernels) per block
    assert line["gpu_launches"] == 3 * (4 * 2 + 2)
