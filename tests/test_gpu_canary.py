"""Guard bands around every buffer (a stand-in for a memory checker, which cannot see a store
past the end of an array when the values inside are right).  w, w_bak, ms, v, out_w and the
gradient pool each live INSIDE a larger tensor with 4 KB of a known pattern on both sides; after
single messages and fused windows of every kind the guards must be untouched, the gradient
pool unchanged, and inside w_bak only [0, n) of each slab (plus, by contract, the slab's
padding) may have changed.  Results are compared with the CPU checker as well."""
from __future__ import annotations

import os

import numpy as np
import pytest

from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

GUARD = 1024                      # floats = 4 KB on each side
PATTERN = -1.2345678e-30          # unlikely to be produced by the update


class Guarded:
    """`count` elements of dtype in the middle of a larger tensor filled with a pattern."""

    def __init__(self, count: int, dtype, pattern):
        import torch
        self.big = torch.full((count + 2 * GUARD,), pattern, dtype=dtype, device="cuda")
        self.view = self.big[GUARD: GUARD + count]
        self.pattern = pattern
        assert self.view.data_ptr() % 16 == 0

    def guards_intact(self) -> bool:
        import torch
        ref = torch.full((GUARD,), self.pattern, dtype=self.big.dtype, device="cuda")
        return bool(torch.equal(self.big[:GUARD], ref)) and bool(torch.equal(self.big[-GUARD:], ref))


SIZES = [5, 1021, 1022, 1023, 1024, 1025, 2047, 2048, 2049, 2050, 2051, 6001]


@pytest.mark.parametrize("vecs", ["1", "2"])
@pytest.mark.parametrize("momentum", [False, True])
@pytest.mark.parametrize("adaptive,bf16", [(True, False), (False, True)])
def test_no_kernel_writes_outside_its_arrays(vecs, momentum, adaptive, bf16, monkeypatch):
    import torch
    monkeypatch.setenv("DCASGD_REPLAY_VECS", vecs)       # read by dcasgd_create: one or two vectors per thread in the fused kernel
    for n in SIZES:                                        # n mod 4 = 0..3; below, at and above one CTA's span (1024 / 2048 elements)
        wl = synth.Workload(name="t", n=n, M=5, pushes=70, adaptive=adaptive, bf16_grad=bf16, eta=0.1,
                            lam=2.0 if adaptive else 0.04, mu=0.95 if adaptive else 0.0, eps=1e-7 if adaptive else 0.0,
                            num_grads=6, nseg=3, sigma_lo_exp=-4, sigma_hi_exp=-1, seed=n)
        ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
        stride, row = B.padded_stride(n), pool.shape[1]
        beta = 0.9 if momentum else None
        for K in (1, 8, 32, 1000):
            w = Guarded(n, torch.float32, PATTERN)
            bak = Guarded(wl.M * stride, torch.float32, PATTERN)
            ms = Guarded(n, torch.float32, PATTERN) if adaptive else None
            vel = Guarded(n, torch.float32, PATTERN) if momentum else None
            out = Guarded(n, torch.float32, PATTERN)
            gp = Guarded(wl.num_grads * row, torch.int16 if bf16 else torch.float32, 12345 if bf16 else PATTERN)
            w.view.copy_(torch.from_numpy(w0))
            host_pool = torch.from_numpy(pool.view(np.int16) if bf16 else pool).reshape(-1)
            gp.view.copy_(host_pool)
            pool_before = gp.big.clone()
            h = B.dcasgd_create(n, wl.M, B.ADAPTIVE if adaptive else B.CONST, B.BF16 if bf16 else B.F32, wl.eta, wl.lam,
                                wl.mu, wl.eps, w.view, bak.view, stride, None if ms is None else ms.view,
                                torch.cuda.current_stream().cuda_stream, v=None if vel is None else vel.view,
                                beta=0.0 if beta is None else beta)
            cpu = U.cpu_server(wl, w0, beta=beta)
            gsz = 2 if bf16 else 4
            B.dcasgd_pull(h, 3, out.view)
            B.dcasgd_push(h, 3, gp.view.data_ptr() + 2 * row * gsz, 0.05)
            cpu.pull(3)
            cpu.push(3, pool[2, :n], np.float32(0.05))
            B.dcasgd_apply_log(h, ev, gp.view, row * gsz, wl.num_grads, K)
            cpu.replay(ev, pool[:, :n])
            B.dcasgd_pull(h, 0, out.view)
            cpu.pull(0)
            torch.cuda.synchronize()
            B.dcasgd_destroy(h)
            what = f"n={n} K={K} V={vecs}"
            for name, g in (("w", w), ("w_bak", bak), ("ms", ms), ("v", vel), ("out_w", out), ("grad_pool", gp)):
                if g is not None:
                    assert g.guards_intact(), f"{what}: a kernel wrote into the guard band of {name}"
            assert torch.equal(gp.big, pool_before), f"{what}: the gradient pool was written"
            same = lambda got, want: np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))
            assert same(w.view, cpu.w) and same(out.view, cpu.w), what
            assert same(bak.view.view(wl.M, stride)[:, :n], cpu.w_bak), what
            if adaptive:
                assert same(ms.view, cpu.ms), what
            if momentum:
                assert same(vel.view, cpu.v), what
            # slab padding: by contract it may be overwritten, and only with whole vectors of the slab's
            # own last elements; beyond the last vector that holds an element it keeps the pattern
            pad = bak.view.view(wl.M, stride)[:, (n + 3) // 4 * 4:].cpu().numpy()
            assert np.all(pad == np.float32(PATTERN)), f"{what}: w_bak padding beyond the last vector was written"
