"""Host-side checks of what bench.py reports without a GPU: the committed ncu traffic summary parses, names the kernels
a call launches, and the reference arm prints the contract's line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_profiled_traffic_matches_the_launch_chain():
    for name, min_bytes in (("c2", 17.0e6), ("c3", 138.9e6), ("c4", 83.8e6)):
        w = bench.make_workload(name)
        total, kernels, src = bench.profiled_traffic(name)
        assert src == os.path.join("profiles", "dram_traffic_per_call.txt")
        assert total is not None and total >= min_bytes                   # DRAM traffic is not below the algorithmic bytes
        assert total < 2.0 * bench.algorithmic_bytes(name, w)
        assert "sonic_stream_kernel" in kernels and "sonic_merge_kernel" in kernels and "sonic_exact_kernel" in kernels
        launches = sum(k["launches_per_call"] for k in kernels.values())
        assert launches == bench.launches_per_call(name, w), (name, launches)
        # the streaming kernel moves the call's bytes
        assert kernels["sonic_stream_kernel"]["dram_bytes_per_call"] >= 0.95 * bench.algorithmic_bytes(name, w)


def test_job_value_is_whole_job_throughput():
    assert bench.job_value(60.0, 1) == 60.0
    assert bench.job_value(60.0, 8) == 7.5       # eight independent replicas finish eight calls per 60 us


def test_reference_arm_prints_the_contract_line():
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--workload", "c1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert run.returncode == 0, run.stderr[-2000:]
    line = json.loads(run.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == "us"
    assert line["higher_is_better"] is False and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"].startswith("c1:")
