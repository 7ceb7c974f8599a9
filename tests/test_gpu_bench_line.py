"""The benchmark's one JSON line on a shrunk workload: the keys the measurement contract names are there, the
numbers hang together, and the GPU arm and the oracle arm describe the same workload."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--config", "dense8b", "--blocks", "2", "--block-len", "512",
           "--decode-steps", "8", "--steps", "2", "--warmup", "3"] + list(extra)
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    return json.loads(r.stdout.strip().splitlines()[-1])


def test_bench_line_has_the_contract_keys_and_consistent_numbers():
    d = _run()
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks",
                "per_config", "phases", "timing"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 2 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["config"]["workload"] == "dense8b" and d["config"]["blocks"] == 2 and d["config"]["decode_steps"] == 8
    tokens = 2 * 8
    assert abs(d["value"] - tokens / (d["ms_per_step"] * 1e-3)) <= 1e-6 * d["value"]
    roof = d["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s"
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    # a shrunk workload has no profiler capture behind it: no traffic is implied
    assert roof["traffic"] is None and roof["traffic_cold"] is None and roof["frac_cold_l2"] is None
    assert d["per_config"] == {}                       # the other configurations are measured in the unmodified run only
    # one prefill launch, bulk append + length advance, one fused launch per decode step, per timed event
    assert d["gpu_launches"] == 2 * (1 + 2 + 8)
    e2e = d["e2e"]
    assert e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0 and e2e["value"] < d["value"]
    cpu = d["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0
    assert d["clocks"].keys() >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_both_arms_describe_the_same_workload():
    ours = _run("--skip-e2e", "--skip-cpu")
    ref = _run("--impl", "reference")
    assert ref["impl"] == "reference" and ref["config"] == ours["config"]
    assert ref["metric"] == ours["metric"] and ref["unit"] == ours["unit"]
    assert ref["e2e"]["h2d_bytes_per_step"] == 0 and ref["cpu_baseline"]["kind"] == "oracle"
