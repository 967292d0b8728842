"""The benchmark's JSON line on the tiny workload: every key the measurement contract names is present and sane."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_tiny_workload_prints_one_complete_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny", "--steps", "3", "--warmup", "3",
                          "--sustained-seconds", "0.3"],
                         cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks",
                "sustained", "quantize_sweep", "tensor_peak_8bit_measured", "roofline_quantize", "fp32_block_scales",
                "e4m3_tensor_scales"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["value"] > 0 and d["vs_baseline"] is None and d["dev_status"] == 0
    assert d["config"]["workload"] == "tiny" and d["data"] == "synthetic"
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["achieved"] > 0 and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["gpu_launches"] == 3 * 9          # three quantizer launches and three two-kernel GEMM calls per step
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    # the back-to-back leg: at least the asked-for time, its own clock record, and a fraction of the sustained peak
    sus = d["sustained"]
    assert sus["seconds"] >= 0.25 and sus["value"] > 0 and sus["steps"] >= 3 and "clocks" in sus and sus["peak"] > 0
    # every leg carries the clocks seen while it ran
    assert "clocks" in d["roofline"] and "clocks" in d["roofline_quantize"] and "clocks" in d["e2e"]
    # Table 1's FP32 block scales beside the headline, with a roofline of their own
    f32 = d["fp32_block_scales"]
    assert f32["scale_fmt"] == "fp32" and f32["roofline"]["frac"] > 0 and f32["dev_status"] == 0
    # the two-level scale format on the FP4 pipe: the uniform grid and the E2M1 baseline grid
    e8 = d["e4m3_tensor_scales"]
    for g in ("uniform_int4", "e2m1_baseline"):
        assert e8[g]["gemm_path"] == "nvf4" and e8[g]["value"] > 0 and e8[g]["dev_status"] == 0 and "clocks" in e8[g]
    # BASELINE config 3 in brief: four sizes, uniform grid and E2M1, RTNE and SR, RHT off and on
    sw = d["quantize_sweep"]
    assert [(e["rows"], e["cols"]) for e in sw] == [(4096, 4096), (8192, 8192), (16384, 8192), (32768, 8192)]
    for e in sw:
        for g in ("int4", "e2m1"):
            for r in ("rtne", "sr"):
                assert e[f"{g}_{r}_rht0"]["gbs"] > 0 and e[f"{g}_{r}_rht16"]["frac"] > 0 and e[f"{g}_{r}_fused_over_standalone"] > 0.5
