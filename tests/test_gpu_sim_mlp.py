"""End-to-end simulated asynchronous training (2-layer MLP, 8 workers, seeded event order):
the server's trajectory on the GPU must equal the CPU checker's after EVERY push, when the
checker is handed the same gradient bytes step by step; and delay compensation must behave as
the paper describes (SGD reference, ASGD = lambda 0, DC-ASGD-a)."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from paper_1609_08326_b200 import sim_mlp, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def data():
    return sim_mlp.make_data(0, "cuda")


@pytest.mark.parametrize("mode", ["sgd", "asgd", "dcasgd-a"])
def test_trajectory_matches_the_checker_after_every_push(mode, data):
    M, pushes, eta = 8, 150, 0.02
    seen = []

    def observer(t, m, g, srv):
        seen.append((m, g.cpu().numpy().copy(), srv.w.cpu().numpy().copy()))

    srv, curve, ev = sim_mlp.run(mode, pushes, M, eta, data=data, observer=observer, eval_every=50)
    adaptive = mode == "dcasgd-a"
    f = np.float32
    cpu = oracle.Server(sim_mlp.init_params(0), M, adaptive, f(eta), f(2.0 if adaptive else 0.0),
                        f(0.95 if adaptive else 0.0), f(1e-7 if adaptive else 0.0))
    t = 0
    for r in ev:
        m = int(r["worker"])
        if r["kind"] == synth.PULL:
            cpu.pull(m)
            continue
        wm, g, w_gpu = seen[t]
        assert wm == m
        cpu.push(m, g, f(r["eta"]))
        assert np.all(np.abs(w_gpu - cpu.w) <= 1e-5 * (1 + np.abs(cpu.w)))
        assert np.array_equal(w_gpu.view(np.uint32), cpu.w.view(np.uint32)), f"w differs after push {t + 1}"
        t += 1
    assert t == pushes == srv.step
    assert np.array_equal(srv.w_bak.cpu().numpy().view(np.uint32), cpu.w_bak.view(np.uint32))
    assert curve[-1][1] < curve[0][1] or curve[0][1] < 0.05          # the loss goes down


def test_modes_relate_as_in_the_paper(data):
    """tau = 0 makes the compensation vanish (DC-ASGD-a on the SGD log equals SGD bit for bit);
    with real delays ASGD and DC-ASGD-a leave the SGD trajectory and differ from each other."""
    import torch
    pushes = 200
    sgd, _, _ = sim_mlp.run("sgd", pushes, data=data)
    asgd, _, _ = sim_mlp.run("asgd", pushes, data=data)
    dca, curve, _ = sim_mlp.run("dcasgd-a", pushes, data=data)
    assert not torch.equal(sgd.w, asgd.w) and not torch.equal(asgd.w, dca.w)
    assert all(np.isfinite(l) for _, l in curve)


# ---- the study of lambda_0 (supplementary material) and checkpoint / resume, on the harder setting

HARD = dict(M=sim_mlp.SWEEP["M"], eta=sim_mlp.SWEEP["eta"], order=sim_mlp.SWEEP["order"],
            order_param=sim_mlp.SWEEP["order_param"])


@pytest.fixture(scope="module")
def hard_data():
    return sim_mlp.make_data(0, "cuda", sim_mlp.SWEEP["noise_std"], normalize=True)


def checker_for(lam0, adaptive=True):
    f = np.float32
    return oracle.Server(sim_mlp.init_params(0), HARD["M"], adaptive, f(HARD["eta"]), f(lam0),
                         f(0.95 if adaptive else 0.0), f(1e-7 if adaptive else 0.0))


def test_lambda0_zero_is_the_asgd_trajectory(hard_data):
    """Too small a lambda_0 degenerates to ASGD; lambda_0 = 0 is ASGD exactly (Section 5's remark
    that ASGD is the lambda = 0 case of DC-ASGD), whatever MeanSquare does meanwhile."""
    import torch
    pushes = 160
    asgd, _, ev = sim_mlp.run("asgd", pushes, data=hard_data, **HARD)
    zero, _, _ = sim_mlp.run("dcasgd-a", pushes, lam0=0.0, data=hard_data, **HARD)
    assert torch.equal(asgd.w, zero.w) and torch.equal(asgd.w_bak, zero.w_bak)
    tau = synth.delays(ev, HARD["M"])
    assert tau.max() >= 20 and tau.mean() >= 5          # the setting really is delay-heavy


@pytest.mark.parametrize("lam0", [0.04, 0.5, 2.0])
def test_sweep_runs_match_the_checker_at_sampled_pushes(lam0, hard_data):
    pushes, every = 150, 25
    seen = []

    def observer(t, m, g, srv):
        seen.append((m, g.cpu().numpy().copy(), srv.w.cpu().numpy().copy() if t % every == 0 or t == pushes else None))

    srv, curve, ev = sim_mlp.run("dcasgd-a", pushes, lam0=lam0, data=hard_data, observer=observer, **HARD)
    cpu, t = checker_for(lam0), 0
    for r in ev:
        m = int(r["worker"])
        if r["kind"] == synth.PULL:
            cpu.pull(m)
            continue
        wm, g, w_gpu = seen[t]
        cpu.push(m, g, np.float32(r["eta"]))
        t += 1
        if w_gpu is not None:
            assert np.all(np.abs(w_gpu - cpu.w) <= 1e-5 * (1 + np.abs(cpu.w)))
            assert np.array_equal(w_gpu.view(np.uint32), cpu.w.view(np.uint32)), f"lambda0={lam0}: w differs after push {t}"
    assert t == pushes and np.array_equal(srv.ms.cpu().numpy().view(np.uint32), cpu.ms.view(np.uint32))
    assert all(np.isfinite(l) for _, l in curve)


def test_resume_in_the_middle_of_training(hard_data):
    """Stop after a pushes, save the server state, continue with a NEW server: the final model
    equals the uninterrupted run's and the checker's, bit for bit."""
    import torch
    pushes, a = 150, 67
    grads = []
    whole, _, ev = sim_mlp.run("dcasgd-a", pushes, data=hard_data,
                               observer=lambda t, m, g, srv: grads.append(g.cpu().numpy().copy()), **HARD)
    first, _, _ = sim_mlp.run("dcasgd-a", pushes, data=hard_data, stop_after=a, **HARD)
    assert first.step == a
    ckpt = first.state_dict()
    first.close()
    del first
    again, _, _ = sim_mlp.run("dcasgd-a", pushes, data=hard_data, state=ckpt, **HARD)
    assert again.step == pushes
    for x, y in ((whole.w, again.w), (whole.w_bak, again.w_bak), (whole.ms, again.ms)):
        assert torch.equal(x, y)
    cpu, t = checker_for(2.0), 0
    for r in ev:
        if r["kind"] == synth.PULL:
            cpu.pull(int(r["worker"]))
        else:
            cpu.push(int(r["worker"]), grads[t], np.float32(r["eta"]))
            t += 1
    assert np.array_equal(again.w.cpu().numpy().view(np.uint32), cpu.w.view(np.uint32))
    assert np.array_equal(again.w_bak.cpu().numpy().view(np.uint32), cpu.w_bak.view(np.uint32))
