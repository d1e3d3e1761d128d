"""The element-range sharded server on CPU: partition bounds, and two gloo ranks that (i) each
replay the log on their own range with the CPU checker and together hold exactly the state of
the whole-vector checker, (ii) reassemble the model with the package's all-gather helper and
(iii) distribute a gradient held by one rank with its scatter helper.  The arithmetic on the
ranks is the checker's (there is no GPU here); what is under test is the package's host logic:
`sharded.partition / gather_model / scatter_gradient`."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_1609_08326_b200 import sharded  # noqa: E402


@pytest.mark.parametrize("n", [0, 1, 31, 32, 33, 1000, 272_474, 25_557_032, 138_357_544])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_partition_covers_the_vector_with_aligned_contiguous_ranges(n, world):
    parts = sharded.partition(n, world)
    c = sharded.chunk_elems(n, world)
    assert c % sharded.ALIGN == 0 and c * world >= n
    assert parts[0][0] == 0 and parts[-1][1] == n
    for r, (lo, hi) in enumerate(parts):
        assert lo <= hi and lo == min(r * c, n) and hi - lo <= c
        assert lo % sharded.ALIGN == 0 or lo == n                 # 128-byte aligned shard starts
        if r:
            assert parts[r - 1][1] == lo                          # contiguous, no gap, no overlap
    sizes = [hi - lo for lo, hi in parts]
    assert all(s == c for s in sizes[: max(0, (n // c))])         # every full shard has exactly chunk elements
    with pytest.raises(ValueError):
        sharded.shard_range(n, world, world)


def test_single_process_helpers_are_the_identity():
    import torch
    w = torch.arange(70, dtype=torch.float32)
    assert torch.equal(sharded.gather_model(w, 70, 1), w)
    assert torch.equal(sharded.scatter_gradient(w, 70, 1, 0, 0), w)


CHILD = r"""
import os, sys
sys.path.insert(0, os.environ["DCASGD_ROOT"])
import numpy as np
import torch
import torch.distributed as dist
import oracle
from paper_1609_08326_b200 import sharded, synth

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
f = np.float32
n = int(os.environ["DCASGD_N"])
wl = synth.Workload(name="t", n=n, M=5, pushes=40, adaptive=True, bf16_grad=False, eta=0.1, lam=2.0, mu=0.95,
                    eps=1e-7, num_grads=7, nseg=3, sigma_lo_exp=-4, sigma_hi_exp=-1, seed=4)
lo, hi = sharded.shard_range(n, world, rank)
ev = wl.log()
sigma, seg = wl.sigma(), wl.seg_len

# every rank draws only its own slice of the inputs (the generator is addressable by element index)
w0 = synth.normal_into(np.empty(hi - lo, dtype=np.float32), lo, wl.seed, synth.STREAM_W0, wl.w0_sigma)
pool = np.stack([synth.normal_into(np.empty(hi - lo, dtype=np.float32), lo, wl.seed, synth.STREAM_GRAD0 + k, sigma, seg)
                 for k in range(wl.num_grads)])
shard = oracle.Server(w0, wl.M, True, f(wl.eta), f(wl.lam), f(wl.mu), f(wl.eps))
shard.replay(ev, pool)

# (ii) the worker's view of the model: all-gather of the shards
full_w = sharded.gather_model(torch.from_numpy(shard.w), n, world, dist).numpy().copy()
full_ms = sharded.gather_model(torch.from_numpy(shard.ms), n, world, dist).numpy().copy()
full_bak = np.stack([sharded.gather_model(torch.from_numpy(np.ascontiguousarray(shard.w_bak[m])), n, world, dist).numpy().copy()
                     for m in range(wl.M)])

# (i) the whole-vector checker, on every rank, must equal the reassembled shards bit for bit
whole = oracle.Server(wl.w0(), wl.M, True, f(wl.eta), f(wl.lam), f(wl.mu), f(wl.eps))
gfull = np.stack([wl.grad(k) for k in range(wl.num_grads)])
whole.replay(ev, gfull)
ok = (np.array_equal(full_w.view(np.uint32), whole.w.view(np.uint32))
      and np.array_equal(full_ms.view(np.uint32), whole.ms.view(np.uint32))
      and np.array_equal(full_bak.view(np.uint32), whole.w_bak.view(np.uint32))
      and np.array_equal(w0, wl.w0()[lo:hi]) and shard.step == whole.step)

# (iii) a full gradient on rank 1 reaches every owner as its slice
src = world - 1
g = torch.from_numpy(gfull[3].copy()) if rank == src else None
recv = torch.empty(sharded.chunk_elems(n, world), dtype=torch.float32)
mine = sharded.scatter_gradient(g, n, world, rank, src, dist, out=recv)
ok = ok and np.array_equal(mine.numpy(), gfull[3][lo:hi])
dist.barrier()
print(f"RESULT {rank} {int(ok)} {lo} {hi}", flush=True)
dist.destroy_process_group()
"""


@pytest.mark.parametrize("n", [10_007, 64, 40])
def test_two_gloo_ranks_shard_the_server(tmp_path, n):
    """n = 40 leaves the second rank a short shard (8 elements); n = 64 fills both exactly."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DCASGD_ROOT=ROOT, DCASGD_N=str(n))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    bounds = sharded.partition(n, 2)
    for rank, (out, _) in enumerate(outs):
        line = [ln for ln in out.splitlines() if ln.startswith("RESULT")][0].split()
        assert int(line[1]) == rank and int(line[2]) == 1
        assert (int(line[3]), int(line[4])) == bounds[rank]
