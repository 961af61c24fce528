"""The benchmark's one JSON line carries every key of its contract (a short run on the GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_bench_line_has_every_contract_key():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5",
                        "--warmup", "3", "--e2e-steps", "1", "--leg-seconds", "0.05"],
                       capture_output=True, text=True, timeout=1500, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # ONE JSON line
    j = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config",
                "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in j, key
    assert j["n_gpus"] == 1 and j["steps"] == 5 and j["warmup"] == 3
    assert j["higher_is_better"] is True and j["scaling"] == "weak" and j["data"] == "synthetic"
    assert j["vs_baseline"] is None
    assert "workload" in j["config"] and "model" not in j["config"]
    assert j["value"] > 0 and j["ms_per_step"] > 0
    assert j["config"]["workload"].startswith("c4")
    assert j["gpu_launches"] == 3 * 5                         # the library's launches, counted
    e2e = j["e2e"]
    assert e2e["h2d_bytes_per_step"] == 16 * 4 * 335_141_888
    assert e2e["d2h_bytes_per_step"] == 2 * 4 * 335_141_888
    assert 0 < e2e["value"] < j["value"]                      # host copies are inside its region
    assert e2e["results_arrived"] is True
    roof = j["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s"
    # the dominant kernel is the call group with the largest measured share of the step
    c4 = j["kernels"]["c4"]
    calls = {"nc_compress_kernel": "nc_compress_batch", "nc_aggregate_kernel": "nc_aggregate",
             "nc_sum_fp32_kernel": "nc_sum_fp32"}
    slowest = max(calls.values(), key=lambda c: c4[c]["ms"])
    assert calls[roof["kernel"].split()[0]] == slowest
    for leg in ("c1", "c2", "c3", "c4", "c5"):
        assert leg in j["kernels"], leg
    assert {"nd_norms_batch", "nd_round_batch", "nd_compress_batch", "nd_aggregate"} <= set(
        j["kernels"]["c3"])
    assert len(j["rooflines"]) >= 12
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-3
    assert roof["traffic"] is None or roof["traffic"] > 0
    cpu = j["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and cpu["sample"]
    assert cpu["one_thread"] > 0
    clocks = j["clocks"]
    assert clocks["sm_max_mhz"] >= clocks["sm_mhz"] > 0 and isinstance(clocks["reasons"], list)
