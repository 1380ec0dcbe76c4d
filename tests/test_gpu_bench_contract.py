"""bench.py prints exactly one JSON line with the keys the benchmark contract names (small case)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    r = subprocess.run([sys.executable, "bench.py", "--gpus", "1", "--steps", "3", "--warmup", "3",
                        "--pool-blocks", "1024", "--request-blocks", "256", "--e2e-steps", "1",
                        "--no-cpu-baseline"], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
              "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "gpu_launches", "roofline",
              "e2e"):
        assert k in d, k
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 3 and d["dtype"] == "u8"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"] == "8b_80k" and "model" not in d["config"]
    assert d["gpu_launches"] == 6                       # one pack and one unpack launch per step
    roof = d["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 1000
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert roof["algorithmic_bytes_per_launch"] == 2 * d["config"]["bytes_each_way"]
    for side in ("pack", "unpack"):                     # jitter is visible in the record itself
        t = roof[side]
        assert t["min_ms"] <= t["median_ms"] <= t["max_ms"] and t["min_ms"] <= t["ms"] <= t["max_ms"]
        assert len(roof["per_step_ms"][side]) == 3
    assert "traffic_source" in roof and roof["traffic"] is None   # not the workload the capture was of
    ov = d["overlap_with_compute"]                      # config 5 in brief, after the timed region
    assert {r["copy_blocks"] for r in ov["runs"]} == {"default", "KVC_PRESET_BESIDE_COMPUTE"}
    assert {r["direction"] for r in ov["runs"]} == {"offload", "load"}
    for r in ov["runs"]:
        assert r["link_gbs_with_gemm"] > 5 and 0.8 < r["gemm_slowdown"] < 2.0
    e2e = d["e2e"]
    assert e2e["h2d_bytes_per_step"] == e2e["d2h_bytes_per_step"] == d["config"]["bytes_each_way"]
    assert 0 < e2e["value"] < d["value"]                # the host link is slower than HBM
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    # 4 x bytes each way per step over the step time
    assert abs(d["value"] - 4 * d["config"]["bytes_each_way"] / (d["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * d["value"]
