"""The benchmark's CPU-only pieces: the reference arm (the CPU checker timed on host cores)
prints one well-formed JSON line, and the log-sampling helpers cut where they should."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_1609_08326_b200 import synth  # noqa: E402


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "c1_resnet20_const", "--steps", "2", "--warmup", "1", "--ref-pushes", "6"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "DC-ASGD element-updates/s" and d["unit"] == "element-updates/s"
    assert d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["dtype"] == "f32" and d["data"] == "synthetic"
    assert d["config"]["workload"] == "c1_resnet20_const" and "sample" in d["config"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_other_ranks_of_the_reference_arm_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_sample_log_keeps_whole_push_pull_pairs():
    import bench
    ev = synth.event_log(4, 50, synth.ORDER_UNIFORM, synth.PROTO_ASYNC, 5, 0.1, seed=0)
    s = bench.sample_log(ev, 7)
    assert int(np.sum(s["kind"] == synth.PUSH)) == 7 and s[-1]["kind"] == synth.PULL
    assert len(bench.sample_log(ev, 10_000)) == len(ev)
    assert bench.row_elems(272_474) % 32 == 0 and bench.row_elems(272_474) >= 272_474


def test_steady_sample_starts_after_the_leading_pulls():
    import bench
    M = 4
    ev = synth.event_log(M, 50, synth.ORDER_UNIFORM, synth.PROTO_ASYNC, 5, 0.1, seed=0)
    s = bench.steady_sample(ev, M, 9)
    assert s[0]["kind"] == synth.PUSH and s[-1]["kind"] == synth.PULL
    assert int(np.sum(s["kind"] == synth.PUSH)) == 9 == int(np.sum(s["kind"] == synth.PULL))
    assert len(bench.steady_sample(ev, M, 10_000)) == len(ev) - M


def test_a_rank_draws_exactly_its_slice_of_the_inputs():
    import bench
    wl = synth.workload("c2_adaptive_1p7m").scaled(n=10_007, num_grads=3, pushes=10)
    w0, pool, view, ev = bench.host_inputs(wl, 2, pin=False)
    lo, hi = 4_992, 10_007
    w0s, pools, views, evs = bench.host_inputs_slice(wl, lo, hi, 2, pin=False)
    assert np.array_equal(w0s.numpy(), w0.numpy()[lo:hi])
    assert np.array_equal(views[:, : hi - lo], view[:, lo:hi])
    assert np.array_equal(evs, ev)
