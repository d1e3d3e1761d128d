"""The benchmark's GPU arm on the smallest workload: one well-formed JSON line with every key
the contract names, for the default (replica) mode and for the sharded mode on one rank."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*flags: str) -> dict:
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "c1_resnet20_const",
                          "--steps", "3", "--warmup", "3", *flags], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def check_common(d: dict, scaling: str) -> None:
    assert d["metric"] == "DC-ASGD element-updates/s" and d["unit"] == "element-updates/s"
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["scaling"] == scaling and d["vs_baseline"] is None and d["dtype"] == "f32" and d["data"] == "synthetic"
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] > 0
    assert d["config"]["workload"] == "c1_resnet20_const" and d["config"]["n"] == 272_474
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["achieved"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["peak_kind"] in ("of measured", "of fallback")
    assert "sm_mhz" in d["clocks"] and "reasons" in d["clocks"]


def test_default_mode_prints_the_contract_line():
    d = run_bench("--no-cpu-baseline")
    check_common(d, "weak")
    assert set(d["variants"]) == {"fused_k8", "fused_k256", "unfused_k1"} and set(d["kernels"]) == {"k_push", "k_pull"}
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 272_474 * 4 * 2000 and e["d2h_bytes_per_step"] == 272_474 * 4
    assert e["value"] < d["value"]                       # host copies are inside the timed region
    # 126 windows of 32 records and one init kernel per step
    assert d["gpu_launches"] == 3 * (d["roofline"]["launches_per_step"] + 1)
    assert "workloads" not in d                          # the other configurations ride with the default workload only


def test_sharded_mode_on_one_rank():
    d = run_bench("--sharded")
    check_common(d, "strong")
    assert d["config"]["shard_elements"] == 272_474 and "shards" in d["config"]["parallelism"]
    assert d["pull_allgather"]["ms"] > 0 and d["pull_allgather"]["model_bytes"] == 272_474 * 4
