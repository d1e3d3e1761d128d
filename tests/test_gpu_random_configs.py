"""Seeded random configurations (sizes from 1 to 1.2 M elements, 1..40 workers, every window size,
protocol, variant, gradient type, momentum on and off, odd hyper-parameters, logs applied in two
pieces): the CUDA library must equal the CPU checker bit for bit on each."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1609_08326_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(6))
def test_random_configurations(seed):
    rng = np.random.default_rng(1000 + seed)
    for case in range(25):
        big = case % 8 == 0                                   # long enough for two vectors per thread
        n = int(rng.integers(600_000, 1_200_000)) if big else int(rng.choice(
            [rng.integers(1, 40), rng.integers(40, 5000), rng.integers(5000, 200_000)]))
        M, G = int(rng.integers(1, 40)), int(rng.integers(1, 12))
        P = int(rng.integers(1, 100 if big else 250))
        adaptive, bf16 = bool(rng.integers(2)), bool(rng.integers(2))
        beta = None if rng.random() < 0.5 else float(rng.choice([0.0, 0.5, 0.9]))
        K = int(rng.choice([1, 2, 3, 5, 8, 16, 32, 64, 200, 1000]))
        wl = synth.Workload(
            name="random", n=n, M=M, pushes=P, adaptive=adaptive, bf16_grad=bf16, eta=float(rng.choice([0.01, 0.1, 0.5])),
            lam=float(rng.choice([2.0, 0.04, 0.0, -1.0])), mu=float(rng.choice([0.0, 0.5, 0.95])) if adaptive else 0.0,
            eps=float(rng.choice([1e-7, 0.0, 1e-3])) if adaptive else 0.0, num_grads=G, nseg=int(rng.integers(1, 5)),
            sigma_lo_exp=-5, sigma_hi_exp=0, seed=int(rng.integers(1 << 30)),
            proto=int(rng.choice([synth.PROTO_ASYNC, synth.PROTO_ASYNC, synth.PROTO_TAU0, synth.PROTO_SYNC])),
            order=int(rng.integers(3)), order_param=1.2)
        ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
        if len(ev) == 0:
            continue
        dpool = U.to_device(pool)
        gpu, cpu = U.gpu_server(wl, w0, beta=beta), U.cpu_server(wl, w0, beta=beta)
        cut = int(rng.integers(0, len(ev) + 1))
        gpu.apply_log(ev[:cut], dpool, K)
        gpu.apply_log(ev[cut:], dpool, int(rng.choice([K, 1, 32])))
        with np.errstate(all="ignore"):
            cpu.replay(ev, pool[:, :n])
        U.assert_state_equal(gpu, cpu, what=f"seed {seed} case {case} {wl} K={K} beta={beta} ")
        gpu.close()
