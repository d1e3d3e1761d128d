"""GPU parity: the CUDA library, called through its C ABI, against the CPU checker on the same
seeded inputs.  The library never fuses a multiply-add and uses IEEE sqrt and division, so the
bar is equality of every bit of w, w_bak[m] and ms (the stated tolerance
max|dw| <= 1e-5 (1+|w|) is asserted as well)."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

PULL, PUSH = B.PULL, B.PUSH


def small_workload(n, adaptive, bf16, M=3, pushes=24, G=6, seed=1, **kw):
    return synth.Workload(name="t", n=n, M=M, pushes=pushes, adaptive=adaptive, bf16_grad=bf16, eta=0.1,
                          lam=2.0 if adaptive else 0.04, mu=0.95 if adaptive else 0.0, eps=1e-7 if adaptive else 0.0,
                          num_grads=G, nseg=3 if n >= 30 else 1, sigma_lo_exp=-4, sigma_hi_exp=-1, seed=seed, **kw)


SIZES = [1, 2, 3, 4, 5, 127, 128, 129, 1023, 1024, 2049, 100_003, 272_474]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("adaptive", [False, True])
@pytest.mark.parametrize("bf16", [False, True])
def test_single_messages(n, adaptive, bf16):
    """dcasgd_pull / dcasgd_push one message at a time, ragged sizes (n mod 4 in 0..3, below,
    at and above a CTA's span)."""
    import torch
    wl = small_workload(n, adaptive, bf16)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
    dpool = U.to_device(pool)
    out_w = torch.empty(n, dtype=torch.float32, device="cuda")
    for r in ev:
        m = int(r["worker"])
        if r["kind"] == PULL:
            gpu.pull(m, out_w)
            cpu.pull(m)
            assert np.array_equal(out_w.cpu().numpy(), cpu.w)          # the model sent back to the worker
        else:
            gpu.push(m, dpool[int(r["grad_id"])], float(r["eta"]))
            cpu.push(m, pool[int(r["grad_id"]), :n], float(r["eta"]))
    U.assert_state_equal(gpu, cpu)
    assert gpu.launches == 1 + len(ev)


@pytest.mark.parametrize("K", [1, 2, 3, 8, 32, 1000])
@pytest.mark.parametrize("n", [5, 1023, 50_001])
@pytest.mark.parametrize("adaptive,bf16", [(False, False), (True, False), (False, True), (True, True)])
def test_apply_log_every_window_size(K, n, adaptive, bf16):
    wl = small_workload(n, adaptive, bf16, M=8, pushes=150, G=12, seed=K)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
    gpu.apply_log(ev, U.to_device(pool), K)
    cpu.replay(ev, np.ascontiguousarray(pool[:, :n]))
    U.assert_state_equal(gpu, cpu, what=f"K={K} ")
    if K == 1:
        assert gpu.launches == 1 + len(ev)
    else:
        assert 2 <= gpu.launches <= 1 + -(-len(ev) // 2) + 2


@pytest.mark.parametrize("proto,order", [(synth.PROTO_TAU0, synth.ORDER_UNIFORM), (synth.PROTO_SYNC, synth.ORDER_UNIFORM),
                                         (synth.PROTO_ASYNC, synth.ORDER_ZIPF), (synth.PROTO_ASYNC, synth.ORDER_ROUND_ROBIN_JITTER)])
def test_other_logs(proto, order):
    wl = small_workload(4099, True, False, M=12, pushes=240, G=7, proto=proto, order=order, order_param=1.2)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    for K in (1, 16, 64):
        gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
        gpu.apply_log(ev, dpool, K)
        cpu.replay(ev, np.ascontiguousarray(pool[:, : wl.n]))
        U.assert_state_equal(gpu, cpu)


def test_record_soup_and_limits():
    """Arbitrary records (repeated pulls, pushes with no pull, per-record eta, default eta), and
    logs that overflow a window's slots, pushes and stores."""
    rng = np.random.default_rng(3)
    M, G, n = 40, 5, 777
    logs = []
    for _ in range(6):
        recs = []
        for _ in range(int(rng.integers(1, 200))):
            if rng.random() < 0.55:
                recs.append((PUSH, int(rng.integers(M)), int(rng.integers(G)), float(rng.choice([-1.0, 0.05, 0.2]))))
            else:
                recs.append((PULL, int(rng.integers(M))))
        logs.append(synth.make_log(recs))
    slots = []
    for k in range(M):
        slots += [(PUSH, k, k % G), (PULL, k)]
    slots += [(PUSH, k, k % G) for k in range(M)]
    logs.append(synth.make_log(slots))
    logs.append(synth.make_log([(PUSH, 0, k % G) for k in range(1500)]))
    logs.append(synth.make_log([(PUSH, 0, 0)] + [(PULL, m % M) for m in range(250)] + [(PUSH, 3, 1)]))
    wl = small_workload(n, True, False, M=M, G=G)
    w0, pool = wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    for ev in logs:
        for K in (7, 1000):
            gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
            gpu.apply_log(ev, dpool, K)
            cpu.replay(ev, np.ascontiguousarray(pool[:, :n]))
            U.assert_state_equal(gpu, cpu)


@pytest.mark.parametrize("adaptive,bf16", [(False, False), (True, True)])
def test_long_windows_take_the_large_program(adaptive, bf16):
    """Windows of several hundred pushes (short vectors: launches are what costs) travel in the
    28 KB form of the window program; more pushes or stores than even that holds cut the window."""
    wl = small_workload(3001, adaptive, bf16, M=4, pushes=1500, G=11, seed=5)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    for K in (600, 1280, 100_000):
        gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
        gpu.apply_log(ev, dpool, K)
        cpu.replay(ev, pool[:, : wl.n])
        U.assert_state_equal(gpu, cpu, what=f"K={K} ")
        progs = B.plan_log(ev, wl.M, K, wl.eta, B.dcasgd_get_window_slot_cap(gpu.h))
        assert gpu.launches == 1 + sum(1 for p in progs if p.n_pushes or p.n_stores)
        assert max(p.n_pushes for p in progs) == min(B.MAX_WINDOW_PUSHES, K // 2)
    # more final pulls than a window can store: 1100 workers all pull after one push
    M = 1100
    wl = small_workload(64, adaptive, bf16, M=M, pushes=4, G=3)
    w0, pool = wl.w0(), U.host_pool(wl)
    ev = synth.make_log([(PUSH, 0, 0)] + [(PULL, m) for m in range(M)] + [(PUSH, 3, 1), (PULL, 7), (PUSH, 1099, 2)])
    gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
    gpu.apply_log(ev, U.to_device(pool), 100_000)
    cpu.replay(ev, pool[:, : wl.n])
    U.assert_state_equal(gpu, cpu)
    assert gpu.launches == 3


def test_apply_log_in_pieces_and_step_counter():
    """Replaying 0..a then a..b equals replaying 0..b; t counts pushes only."""
    wl = small_workload(30_001, True, False, M=5, pushes=100, G=9)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
    assert gpu.step == 0
    a = 77
    gpu.apply_log(ev[:a], dpool, 32)
    assert gpu.step == int(np.sum(ev["kind"][:a] == PUSH))
    gpu.apply_log(ev[a:a], dpool, 32)                       # empty log: no-op
    gpu.apply_log(ev[a:], dpool, 5)
    cpu.replay(ev, np.ascontiguousarray(pool[:, : wl.n]))
    U.assert_state_equal(gpu, cpu)
    assert gpu.step == 100


def test_empty_model_and_side_stream():
    import torch
    wl = small_workload(0, True, False)
    srv = B.Server(np.zeros(0, dtype=np.float32), 3, True, 0.1, 2.0, 0.95, 1e-7)
    srv.pull(1)
    srv.push(1, None)
    srv.apply_log(wl.log(), torch.empty((6, 0), device="cuda"), 8, grad_stride_bytes=0, num_grads=6)
    assert srv.step == 1 + wl.pushes and srv.launches == 0
    # a server bound to a non-default stream
    st = torch.cuda.Stream()
    wl = small_workload(12_345, False, False)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    torch.cuda.synchronize()
    gpu, cpu = U.gpu_server(wl, w0, stream=st), U.cpu_server(wl, w0)
    gpu.apply_log(ev, dpool, 16)
    st.synchronize()
    cpu.replay(ev, np.ascontiguousarray(pool[:, : wl.n]))
    U.assert_state_equal(gpu, cpu)


def test_side_stream_with_device_w0_and_resumed_state():
    """The binding fills w (and, on resume, w_bak / ms) on torch's current stream while the
    server's kernels run on its own stream: the first kernel must wait for those copies."""
    import torch
    wl = small_workload(300_007, True, False, M=5, pushes=60, G=9)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    cpu = U.cpu_server(wl, w0)
    cpu.replay(ev, pool[:, : wl.n])
    st = torch.cuda.Stream()
    w0_dev = torch.from_numpy(w0).cuda()
    torch.cuda.synchronize()
    busy = torch.empty(64 << 20, device="cuda")
    for _ in range(20):
        busy.normal_()                                   # keeps the current stream busy ahead of the copies
    gpu = B.Server(w0_dev * 1.0, wl.M, wl.adaptive, wl.eta, wl.lam, wl.mu, wl.eps, stream=st)
    a = 41
    gpu.apply_log(ev[:a], dpool, 16)
    ckpt = gpu.state_dict()
    for _ in range(20):
        busy.normal_()
    resumed = B.Server(None, wl.M, wl.adaptive, wl.eta, wl.lam, wl.mu, wl.eps, stream=st,
                       state={k: (v.cuda() if hasattr(v, "cuda") else v) for k, v in ckpt.items()})
    resumed.apply_log(ev[a:], dpool, 16)
    st.synchronize()
    U.assert_state_equal(resumed, cpu)


def test_errors_leave_the_state_untouched():
    import torch
    wl = small_workload(1000, True, False, M=4)
    w0, pool = wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    gpu = U.gpu_server(wl, w0)
    torch.cuda.synchronize()
    before = (gpu.w.clone(), gpu.w_bak_buf.clone(), gpu.ms.clone())
    launches = gpu.launches

    def expect(status, fn):
        with pytest.raises(B.DcasgdError) as e:
            fn()
        assert e.value.status == status, e.value

    expect(B.EWORKER, lambda: gpu.pull(4))
    expect(B.EWORKER, lambda: gpu.push(9, dpool[0]))
    expect(B.EINVAL, lambda: gpu.push(0, None))
    expect(B.EALIGN, lambda: gpu.push(0, dpool[0].data_ptr() + 4))
    expect(B.EINVAL, lambda: gpu.push(0, gpu.w))                                  # gradient aliases the model
    expect(B.EINVAL, lambda: gpu.push(0, gpu.w_bak_buf[1024:]))
    expect(B.EINVAL, lambda: gpu.push(0, dpool[0], float("nan")))
    expect(B.EINVAL, lambda: gpu.pull(0, gpu.ms))
    good = [(PUSH, 0, 0), (PULL, 0), (PUSH, 1, 1)]
    for bad in ([(PUSH, 4, 0)], [(PUSH, 0, 6)], [(3, 0, 0)], [(PUSH, 0, 0, float("inf"))]):
        for K in (1, 8):
            expect(B.ELOG, lambda: gpu.apply_log(synth.make_log(good + bad), dpool, K))   # bad record at the END
    expect(B.EINVAL, lambda: gpu.apply_log(synth.make_log(good), dpool, 0))
    expect(B.EALIGN, lambda: gpu.apply_log(synth.make_log(good), dpool, 8, grad_stride_bytes=4004))
    expect(B.EINVAL, lambda: gpu.apply_log(synth.make_log(good), gpu.w_bak_buf, 8, grad_stride_bytes=4096, num_grads=2))
    torch.cuda.synchronize()
    assert gpu.launches == launches and gpu.step == 0
    for a, b in zip(before, (gpu.w, gpu.w_bak_buf, gpu.ms)):
        assert torch.equal(a, b)
    # per-call buffers that are not device memory of the server's GPU, or shorter than the call
    # needs, are refused on the host: nothing is launched, so no bad address ever reaches a kernel
    host_g = torch.zeros(1024).pin_memory()
    plain = np.zeros(1024, dtype=np.float32)
    expect(B.EINVAL, lambda: gpu.push(0, host_g))
    expect(B.EINVAL, lambda: gpu.push(0, plain))
    expect(B.EINVAL, lambda: gpu.pull(0, host_g))
    expect(B.EINVAL, lambda: gpu.apply_log(synth.make_log(good[:2]), host_g, 8, grad_stride_bytes=4096, num_grads=1))
    try:                                                 # an allocation of exactly 4000 bytes, outside torch's pools
        from cuda.bindings import runtime as cudart
    except ImportError:
        cudart = None
    if cudart is not None:
        err, raw = cudart.cudaMalloc(4000)
        assert int(err) == 0
        try:
            gpu_ok = U.gpu_server(wl, w0)
            torch.cuda.synchronize()
            n_before = gpu_ok.launches
            gpu_ok.push(0, int(raw))                     # 1000 floats fit exactly
            assert gpu_ok.launches == n_before + 1
            expect(B.EINVAL, lambda: gpu_ok.push(0, int(raw) + 2048))        # 1952 bytes left: too short
            expect(B.EINVAL, lambda: gpu_ok.pull(0, int(raw) + 2048))
            expect(B.EINVAL, lambda: gpu_ok.apply_log(synth.make_log(good), int(raw), 8, grad_stride_bytes=4000, num_grads=2))
            gpu_ok.apply_log(synth.make_log(good[:2]), int(raw), 8, grad_stride_bytes=4000, num_grads=1)   # exactly one buffer fits
            assert gpu_ok.launches == n_before + 2
            torch.cuda.synchronize()
        finally:
            cudart.cudaFree(raw)
    counter = torch.zeros(2, dtype=torch.int64, device="cuda")
    expect(B.EALIGN, lambda: B.dcasgd_check_adaptive_lambda(2.0, 1.0, 2.0, counter.data_ptr() + 4))
    expect(B.EINVAL, lambda: B.dcasgd_check_adaptive_lambda(2.0, 1.0, 2.0, np.zeros(1, dtype=np.int64)))
    torch.cuda.synchronize()
    assert gpu.launches == launches and gpu.step == 0 and int(counter.sum().item()) == 0
    # host memory handed in as state is refused
    host = torch.zeros(1000)
    with pytest.raises(B.DcasgdError):
        B.dcasgd_create(1000, 1, B.CONST, B.F32, 0.1, 0.04, 0, 0, host.data_ptr(), dpool.data_ptr(), 1024, None)


def test_special_values_propagate_like_ieee():
    """inf / nan / denormal / signed-zero inputs: same bits as the checker (no flush to zero)."""
    n = 64
    wl = small_workload(n, True, False, M=2, pushes=6, G=3)
    w0 = wl.w0()
    pool = U.host_pool(wl)
    w0[:8] = [0.0, -0.0, 1e-40, -1e-40, np.inf, -np.inf, np.nan, 3e38]
    pool[0, :8] = [1e-30, -1e-30, 1e-20, 0.0, 1.0, 1e20, 1.0, 3e38]
    pool[1, 8:12] = [np.inf, np.nan, 1e-45, -0.0]
    ev = wl.log()
    for K in (1, 8):
        gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
        gpu.apply_log(ev, U.to_device(pool), K)
        with np.errstate(all="ignore"):
            cpu.replay(ev, np.ascontiguousarray(pool[:, :n]))
        U.assert_state_equal(gpu, cpu)


@pytest.mark.parametrize("lam,eps", [(2.0, 0.0), (0.0, 1e-7), (-0.0, 1e-7), (-2.0, 1e-7), (1e25, 1e-7), (3e-30, 0.0),
                                     (2.0, 1e-38), (0.04, 1e30)])
def test_adaptive_lambda_routes(lam, eps):
    """lambda_t = lambda_0 / sqrt(ms + eps) takes a branch-free exact route when ms + eps lies in
    [2^-100, 2^100) and |lambda_0| in [2^-60, 2^60), and the guarded IEEE route otherwise (zero,
    denormal, huge, non-finite).  Both must give the checker's bits; mixed within one vector."""
    n = 4096
    wl = small_workload(n, True, False, M=4, pushes=40, G=8).scaled(lam=lam, eps=eps)
    w0, pool, ev = wl.w0(), U.host_pool(wl), wl.log()
    rng = np.random.default_rng(5)
    scale = rng.choice([0.0, 1e-30, 1e-22, 1e-12, 1e-3, 1.0, 1e12, 1e18], size=n).astype(np.float32)
    pool[:, :n] = (pool[:, :n] / np.float32(1e-2)) * scale          # every magnitude class in every vector
    for K in (1, 32):
        gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
        gpu.apply_log(ev, U.to_device(pool), K)
        with np.errstate(all="ignore"):
            cpu.replay(ev, pool[:, :n])
        U.assert_state_equal(gpu, cpu, what=f"lam={lam} eps={eps} K={K} ")


def lambda0_cases() -> list[float]:
    """Numerators for the exhaustive-in-s comparison: the paper's settings, powers of two and their
    neighbours one ulp away, all-ones significands, both ends of [2^-60, 2^60), and seeded random
    values spread log-uniformly over that range with random signs."""
    f = np.float32
    vals = [2.0, 0.04, 1.0, -2.0, 0.3, 1.9999999, 7.7e-12, 3.3e9]
    for k in (-60, -31, -1, 0, 1, 24, 59):
        p2 = f(2.0) ** f(k)
        vals += [float(p2), float(np.nextafter(p2, f(np.inf)))]
        if k > -60:
            vals.append(float(np.nextafter(p2, f(0))))               # all-ones significand just below the power of two
    vals.append(float(np.nextafter(f(2.0) ** f(60), f(0))))          # the largest admissible numerator
    rng = np.random.default_rng(20240607)
    mag = np.exp2(rng.uniform(-60, 60, size=40)).astype(f)
    sign = rng.choice([-1.0, 1.0], size=40).astype(f)
    vals += [float(v) for v in mag * sign]
    vals = [v for v in vals if 2.0 ** -60 <= abs(v) < 2.0 ** 60]
    assert len(vals) >= 64
    return vals


def test_adaptive_lambda_branch_free_route_is_exact_for_every_s():
    """For 69 numerators lambda_0 (see lambda0_cases) the branch-free lambda_0 / sqrt(s) equals
    the IEEE sqrt-then-divide on all 1.68e9 binary32 values of s in [2^-100, 2^100)."""
    import torch
    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    last = float(np.nextafter(np.float32(2.0 ** 100), np.float32(0)))
    for lam0 in lambda0_cases():
        B.dcasgd_check_adaptive_lambda(lam0, 2.0 ** -100, last, counter)
    torch.cuda.synchronize()
    assert int(counter.item()) == 0
    for bad in (lambda: B.dcasgd_check_adaptive_lambda(0.0, 1.0, 2.0, counter),
                lambda: B.dcasgd_check_adaptive_lambda(2.0, 0.0, 2.0, counter),
                lambda: B.dcasgd_check_adaptive_lambda(2.0, 1.0, 2.0, None)):
        with pytest.raises(B.DcasgdError):
            bad()


def test_adaptive_lambda_on_a_grid_of_significand_pairs():
    """Numerators and radicands together.  The branch-free route is invariant under scaling the
    numerator by 2 and s by 4, so numerators in [1, 2) and s in [1, 4) stand for all exponents.
    Always: 2^15 numerators strided over all significands (odd stride: low bits vary too) times
    every s in [1, 4) = 5.5e11 pairs, plus every numerator against the radicands whose root has an
    all-ones significand (the one hard case of the reciprocal refinement).
    With DCASGD_EXHAUSTIVE=1: ALL 2^23 x 2^24 = 1.4e14 pairs (a minute or two)."""
    import os

    import torch
    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    below4 = float(np.nextafter(np.float32(4.0), np.float32(0)))
    B.dcasgd_check_adaptive_lambda_grid(1.0, 1 << 15, 255, 1.0, below4, counter)
    hard = float(np.nextafter(np.nextafter(np.float32(4.0), np.float32(0)), np.float32(0)))     # sqrt rounds to 2 - 2^-23
    B.dcasgd_check_adaptive_lambda_grid(1.0, 1 << 23, 1, hard, below4, counter)
    B.dcasgd_check_adaptive_lambda_grid(-1.0, 1 << 23, 1, hard, below4, counter)
    if os.environ.get("DCASGD_EXHAUSTIVE") == "1":
        B.dcasgd_check_adaptive_lambda_grid(1.0, 1 << 23, 1, 1.0, below4, counter)
    torch.cuda.synchronize()
    assert int(counter.item()) == 0
    with pytest.raises(B.DcasgdError):
        B.dcasgd_check_adaptive_lambda_grid(2.0 ** 59, 1 << 23, 2, 1.0, 2.0, counter)       # numerators reach 2^60
    with pytest.raises(B.DcasgdError):
        B.dcasgd_check_adaptive_lambda_grid(1.0, 4, 1, 0.0, 2.0, counter)
    with pytest.raises(B.DcasgdError):
        B.dcasgd_check_adaptive_lambda_grid(1.0, 4, 1, 1.0, 2.0, None)
    B.dcasgd_check_adaptive_lambda_grid(1.0, 0, 1, 1.0, 2.0, counter)                        # nothing to do


def test_apply_log_from_host_overlapped_copies():
    """The pool arrives from pinned host memory on a copy stream while earlier pieces of the log
    replay: same bits as the checker (and as a resident pool)."""
    import torch
    wl = small_workload(200_003, True, False, M=6, pushes=300, G=20)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    host = torch.from_numpy(pool).pin_memory()
    dev = torch.full(host.shape, float("nan"), device="cuda")          # nothing resident beforehand
    gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
    nbytes = B.apply_log_from_host(gpu.h, ev, host, dev, 32, torch.cuda.Stream(), chunk=3)
    assert nbytes == host.numel() * 4
    cpu.replay(ev, pool[:, : wl.n])
    U.assert_state_equal(gpu, cpu)


def test_checkpoint_and_resume():
    """Replay 0..a, save the server state, resume a NEW server from the copy and replay a..b:
    bit for bit the same as replaying 0..b in one go (and as the checker)."""
    wl = small_workload(20_001, True, False, M=5, pushes=120, G=9)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    a = 101
    first = U.gpu_server(wl, w0)
    first.apply_log(ev[:a], dpool, 16)
    ckpt = first.state_dict()
    first.close()
    del first
    resumed = B.Server(None, wl.M, wl.adaptive, wl.eta, wl.lam, wl.mu, wl.eps, wl.bf16_grad, state=ckpt)
    assert resumed.step == ckpt["t"] == int(np.sum(ev["kind"][:a] == PUSH))
    resumed.apply_log(ev[a:], dpool, 16)
    cpu = U.cpu_server(wl, w0)
    cpu.replay(ev, pool[:, : wl.n])
    U.assert_state_equal(resumed, cpu)


def test_delay_compensated_synchronous_rounds():
    """Supplementary: rounds of M pushes against one shared snapshot with eta_hat / M, as a log."""
    M = 8
    wl = small_workload(33_333, False, False, M=M, pushes=M * 12, G=M * 12, proto=synth.PROTO_SYNC).scaled(eta=0.5 / M, lam=2.0)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    for K in (1, 2 * M, 64):
        gpu, cpu = U.gpu_server(wl, w0), U.cpu_server(wl, w0)
        gpu.apply_log(ev, U.to_device(pool), K)
        cpu.replay(ev, pool[:, : wl.n])
        U.assert_state_equal(gpu, cpu)
    (p,) = B.plan_log(ev[: 2 * M], M, 2 * M, wl.eta)
    assert p.n_slots == 1 and p.n_snapshot_reads == 0 and p.n_stores == M      # one shared in-window snapshot


@pytest.mark.parametrize("K", [1, 8, 32, 1000])
@pytest.mark.parametrize("n", [3, 1023, 70_001])
@pytest.mark.parametrize("adaptive,bf16", [(False, False), (True, False), (False, True), (True, True)])
def test_momentum_variant(K, n, adaptive, bf16):
    """Momentum variant (v = beta*v + eta*u ; w = w - v): single messages and fused windows equal
    the checker bit for bit, velocity included; beta = 0 equals the server without momentum."""
    wl = small_workload(n, adaptive, bf16, M=6, pushes=90, G=10, seed=K)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    gpu, cpu = U.gpu_server(wl, w0, beta=0.9), U.cpu_server(wl, w0, beta=0.9)
    gpu.pull(1)
    gpu.push(1, dpool[2], 0.05)
    cpu.pull(1)
    cpu.push(1, pool[2, :n], np.float32(0.05))
    gpu.apply_log(ev, dpool, K)
    cpu.replay(ev, pool[:, :n])
    U.assert_state_equal(gpu, cpu, what=f"momentum K={K} ")
    zero, plain = U.gpu_server(wl, w0, beta=0.0), U.gpu_server(wl, w0)
    zero.apply_log(ev, dpool, K)
    plain.apply_log(ev, dpool, K)
    import torch
    torch.cuda.synchronize()
    assert torch.equal(zero.w, plain.w) and torch.equal(zero.w_bak, plain.w_bak)


def test_momentum_checkpoint_carries_the_velocity():
    wl = small_workload(9_001, True, False, M=4, pushes=60, G=7)
    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    first = U.gpu_server(wl, w0, beta=0.5)
    first.apply_log(ev[:51], dpool, 16)
    ckpt = first.state_dict()
    resumed = B.Server(None, wl.M, wl.adaptive, wl.eta, wl.lam, wl.mu, wl.eps, wl.bf16_grad, state=ckpt, beta=0.5)
    resumed.apply_log(ev[51:], dpool, 16)
    cpu = U.cpu_server(wl, w0, beta=0.5)
    cpu.replay(ev, pool[:, : wl.n])
    U.assert_state_equal(resumed, cpu)
