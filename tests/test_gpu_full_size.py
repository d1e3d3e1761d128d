"""GPU parity at the full sizes of the benchmark workloads, in the launch configurations that
bench.py times (fused windows of 8, 32 and 256 records, 1280 records on the short vectors, and
one kernel per message).

The CPU checker replays the FULL log on a sample of elements (head and tail of the vector, the
neighbourhood of every gradient-scale segment boundary, and a regular stride): elements never
interact, so each sampled output is exactly what the checker gives for the whole vector.  Where
it finishes in seconds it also replays the full vector (all of c1; a 64-push prefix of c3)."""
from __future__ import annotations

import os

import numpy as np
import pytest

from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def sampled_check(wl, w0, pool, dpool, ev, window_ks):
    idx = U.sample_indices(wl.n, wl.seg_len, wl.nseg)
    cpu = U.cpu_server(wl, w0[idx])
    cpu.replay(ev, np.ascontiguousarray(pool[:, idx]))
    for K in window_ks:
        gpu = U.gpu_server(wl, w0)
        gpu.apply_log(ev, dpool, K)
        U.assert_state_equal(gpu, cpu, idx, what=f"{wl.name} K={K} ")
        gpu.close()


def test_c1_resnet20_constant_full_vector_full_log():
    wl = synth.workload("c1_resnet20_const")
    w0, pool, ev = wl.w0(), U.host_pool(wl), wl.log()
    assert len(ev) == 4 + 2 * 2000 and pool.shape[0] == 2000
    dpool = U.to_device(pool)
    servers, bounds = U.cpu_replay_ranges(wl, ev, w0, pool, os.cpu_count() or 1)
    for K in (32, 8, 256, 1280, 1):
        gpu = U.gpu_server(wl, w0)
        gpu.apply_log(ev, dpool, K)
        U.assert_ranges_equal(gpu, servers, bounds)
        gpu.close()


def test_c2_adaptive_full_log_sampled():
    wl = synth.workload("c2_adaptive_1p7m")
    w0, pool, ev = wl.w0(), U.host_pool(wl), wl.log()
    sampled_check(wl, w0, pool, U.to_device(pool), ev, (32, 8, 256, 1280, 1))


def test_c3_resnet50_adaptive_as_benchmarked():
    wl = synth.workload("c3_resnet50_adaptive")
    w0, pool, ev = wl.w0(), U.host_pool(wl), wl.log()
    dpool = U.to_device(pool)
    sampled_check(wl, w0, pool, dpool, ev, (32, 8, 256, 1))
    # full vector on the first 64 pushes
    prefix = ev[: wl.M + 2 * 64]
    servers, bounds = U.cpu_replay_ranges(wl, prefix, w0, pool, os.cpu_count() or 1)
    gpu = U.gpu_server(wl, w0)
    gpu.apply_log(prefix, dpool, 32)
    U.assert_ranges_equal(gpu, servers, bounds)


@pytest.mark.parametrize("name", ["c4_vgg16_const_bf16", "c4_vgg16_adaptive_bf16"])
def test_c4_vgg16_bf16_full_log_sampled(name):
    wl = synth.workload(name)
    w0, pool, ev = wl.w0(), U.host_pool(wl), wl.log()
    assert pool.dtype == np.uint16
    sampled_check(wl, w0, pool, U.to_device(pool), ev, (32, 8, 1))
