"""The element-range sharded server on ONE GPU: the ranks of a 2- and a 3-way partition are
driven one after the other by this process (each is the unchanged server library over its own
range, no collective involved in the update), and the concatenation of their states must equal
the whole-vector CPU checker bit for bit."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1609_08326_b200 import sharded, synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("adaptive,bf16", [(True, False), (False, True)])
def test_shards_back_to_back_equal_the_whole_vector_checker(world, adaptive, bf16):
    import torch
    n = 200_003
    wl = synth.Workload(name="t", n=n, M=6, pushes=80, adaptive=adaptive, bf16_grad=bf16, eta=0.1,
                        lam=2.0 if adaptive else 0.04, mu=0.95 if adaptive else 0.0, eps=1e-7 if adaptive else 0.0,
                        num_grads=9, nseg=5, sigma_lo_exp=-4, sigma_hi_exp=-1, seed=7)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    cpu = U.cpu_server(wl, w0)
    cpu.pull(2)
    cpu.push(2, pool[4, :n], np.float32(0.05))
    cpu.replay(ev, pool[:, :n])

    got_w, got_bak, got_ms = [], [], []
    gathered = torch.empty(world * sharded.chunk_elems(n, world), dtype=torch.float32, device="cuda")
    for rank in range(world):
        lo, hi = sharded.shard_range(n, world, rank)
        assert lo % 32 == 0
        # this rank's columns of the pool, in a buffer of its own (rows padded to 32 elements)
        cols = np.zeros((wl.num_grads, U.row_elems(hi - lo)), dtype=pool.dtype)
        cols[:, : hi - lo] = pool[:, lo:hi]
        dcols = U.to_device(cols)
        srv = sharded.ShardedServer(w0[lo:hi], n, rank, world, wl.M, adaptive, wl.eta, wl.lam, wl.mu, wl.eps, bf16)
        assert (srv.lo, srv.hi) == (lo, hi)
        srv.pull(2)
        srv.push(2, dcols[4], 0.05)
        srv.apply_log(ev, dcols, 32)
        torch.cuda.synchronize()
        assert srv.step == cpu.step
        got_w.append(srv.local.w.cpu().numpy())
        got_bak.append(srv.local.w_bak.cpu().numpy())
        if adaptive:
            got_ms.append(srv.local.ms.cpu().numpy())
        # what the all-gather does on several GPUs, spelled out for one: shard r lands at r*chunk
        gathered[rank * srv.chunk: rank * srv.chunk + (hi - lo)].copy_(srv.local.w)
        srv.close()
    w = np.concatenate(got_w)
    assert np.array_equal(w.view(np.uint32), cpu.w.view(np.uint32))
    assert np.array_equal(np.concatenate(got_bak, axis=1).view(np.uint32), cpu.w_bak.view(np.uint32))
    if adaptive:
        assert np.array_equal(np.concatenate(got_ms).view(np.uint32), cpu.ms.view(np.uint32))
    assert np.array_equal(gathered[:n].cpu().numpy().view(np.uint32), cpu.w.view(np.uint32))


def test_one_rank_world_is_the_plain_server():
    """world = 1: gather and scatter are the identity, the shard is the whole vector."""
    import torch
    wl = synth.Workload(name="t", n=5_001, M=3, pushes=20, adaptive=True, bf16_grad=False, eta=0.1, lam=2.0, mu=0.95,
                        eps=1e-7, num_grads=4, nseg=1, sigma_lo_exp=-2, sigma_hi_exp=-2, seed=1)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    srv = sharded.ShardedServer(w0, wl.n, 0, 1, wl.M, True, wl.eta, wl.lam, wl.mu, wl.eps)
    cpu = U.cpu_server(wl, w0)
    srv.push_from(1, dpool[2][: wl.n], src=0)
    cpu.push(1, pool[2, : wl.n])
    srv.apply_log(ev, dpool, 8)
    cpu.replay(ev, pool[:, : wl.n])
    model = srv.pull(0, gather=True)
    cpu.pull(0)
    torch.cuda.synchronize()
    assert np.array_equal(model.cpu().numpy().view(np.uint32), cpu.w.view(np.uint32))
    U.assert_state_equal(srv.local, cpu)
