"""The N>1 path of the benchmark (independent replicas, one per rank) on CPU: two gloo ranks
aggregate their timings the way bench.py does - slowest rank's time, units summed."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, os.environ["DCASGD_ROOT"])
import torch.distributed as dist
from paper_1609_08326_b200 import accounting
dist.init_process_group("gloo")
rank = dist.get_rank()
ms, units = accounting.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), dist)
dist.barrier()
print(f"RESULT {rank} {ms} {units}", flush=True)
dist.destroy_process_group()
"""


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DCASGD_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    for rank, (out, _) in enumerate(outs):
        line = [ln for ln in out.splitlines() if ln.startswith("RESULT")][0].split()
        assert int(line[1]) == rank
        assert float(line[2]) == 15.0            # max over ranks
        assert float(line[3]) == 3000.0          # units summed


def test_single_process_passthrough():
    from paper_1609_08326_b200 import accounting
    assert accounting.aggregate_over_ranks(12.5, 7.0, None) == (12.5, 7.0)


def test_byte_accounting():
    from paper_1609_08326_b200 import accounting as A
    assert (A.pull_bytes(), A.push_bytes(False, False), A.push_bytes(False, True)) == (8, 16, 14)
    assert (A.push_bytes(True, False), A.push_bytes(True, True)) == (24, 22)
    assert A.unfused_log_bytes(1, 1, True, False) == 32 and A.unfused_log_bytes(1, 1, False, False) == 24

    class P:
        n_pushes, n_stores, n_snapshot_reads = 16, 16, 16
    assert A.window_bytes(P, True, False) == 16 + 64 + 64 + 64       # 208 B per 16-push window
    assert A.window_bytes(P, False, True) == 8 + 32 + 64 + 64
    P.n_pushes = P.n_stores = 0
    assert A.window_bytes(P, True, False) == 0
