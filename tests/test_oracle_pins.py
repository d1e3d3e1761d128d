"""Pins for the CPU checker: what the paper and the mathematics fix, independent of the checker.

Each `pin_*` function takes the checker's shared library, so that the same battery can be run
against deliberately broken copies of the checker (test_oracle_mutants.py) to show that a
plausible mistake anywhere in it fails at least one pin.
"""
from __future__ import annotations

import json
import math
import os
from fractions import Fraction as Fr

import numpy as np
import pytest

import oracle
from paper_1609_08326_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq10_hand_examples.json")
PULL, PUSH = synth.PULL, synth.PUSH


def _golden():
    with open(GOLDEN) as f:
        return json.load(f)


# ------------------------------------------------------------------ exact rational definitions

def eq10_exact(w, wb, g, eta, lam):
    """Section 4, Eq. 10, over the rationals."""
    return w - eta * (g + lam * g * g * (w - wb))


def replay_exact(w0, M, ev, grads, eta, lam):
    """Algorithm 2 over the rationals (constant lambda), element by element."""
    n = len(w0)
    w = [Fr(x) for x in w0]
    wb = [[Fr(x) for x in w0] for _ in range(M)]
    for r in ev:
        m = int(r["worker"])
        if r["kind"] == PULL:
            wb[m] = list(w)
        else:
            g = grads[int(r["grad_id"])]
            e = Fr(float(r["eta"])) if r["eta"] >= 0 else eta
            w = [eq10_exact(w[i], wb[m][i], Fr(float(g[i])), e, lam) for i in range(n)]
    return w, wb


# ------------------------------------------------------------------------------------ pins

def pin_hand_constant(L):
    """Eq. 10 on a 3-element example whose values are exact in binary32."""
    ex = _golden()["constant_lambda"]
    eta, lam = Fr(ex["eta"]), Fr(ex["lambda"])
    want = [eq10_exact(Fr(w), Fr(b), Fr(g), eta, lam) for w, b, g in zip(ex["w"], ex["w_bak"], ex["g"])]
    assert [float(x) for x in want] == ex["expected_w"]           # the stored values are Eq. 10's
    for dt in (np.float32, np.float64):
        s = oracle.Server(ex["w_bak"], 1, False, ex["eta"], ex["lambda"], dtype=dt, library=L)
        s.w[:] = ex["w"]                                         # the model moved on after the pull
        s.push(0, np.asarray(ex["g"], dtype=dt))
        assert s.w.tolist() == ex["expected_w"]
        assert s.w_bak[0].tolist() == ex["w_bak"]                 # a push never touches the backup
        assert s.step == 1


def pin_closed_form_repeated(L):
    """n pushes of one gradient against one snapshot: w_n = w* + (1-a)^n (w_0 - w*)."""
    ex = _golden()["repeated_pushes_one_snapshot"]
    eta, lam, g, wb, w0 = (Fr(ex[k]) for k in ("eta", "lambda", "g", "w_bak", "w0"))
    a = eta * lam * g * g
    wstar = wb - 1 / (lam * g)
    want = [float(wstar + (1 - a) ** n * (w0 - wstar)) for n in (1, 2, 3)]
    assert want == ex["expected_w"]
    s = oracle.Server([ex["w_bak"]], 1, False, ex["eta"], ex["lambda"], dtype=np.float32, library=L)
    s.w[0] = ex["w0"]
    got = []
    for _ in range(3):
        s.push(0, np.asarray([ex["g"]], dtype=np.float32))
        got.append(float(s.w[0]))
    assert got == ex["expected_w"]
    # general (non-dyadic) values, binary64: the geometric closed form within rounding
    rng = np.random.default_rng(5)
    for _ in range(20):
        eta_, lam_, g_, wb_, w0_ = 0.3, 0.7, float(rng.normal()), float(rng.normal()), float(rng.normal())
        a_ = eta_ * lam_ * g_ * g_
        ws_ = wb_ - 1.0 / (lam_ * g_)
        s = oracle.Server([wb_], 1, False, eta_, lam_, dtype=np.float64, library=L)
        s.w[0] = w0_
        for n in range(1, 41):
            s.push(0, np.asarray([g_], dtype=np.float64))
            ref = ws_ + (1.0 - a_) ** n * (w0_ - ws_)
            assert abs(s.w[0] - ref) <= 1e-11 * (1 + abs(ref) + abs(ws_))


def pin_hand_adaptive(L):
    """MeanSquare rule + Eq. 10 on an example where the root and the quotient are exact."""
    ex = _golden()["adaptive"]
    # re-derive the stored trace exactly: ms, lambda_t and w are rationals here
    mu, lam0, eta = Fr(ex["mu"]), Fr(ex["lambda0"]), Fr(ex["eta"])
    ms, w, wb = Fr(0), Fr(ex["w0"]), Fr(ex["w_bak"])
    for p in ex["pushes"]:
        g = Fr(p["g"])
        ms = mu * ms + (1 - mu) * g * g
        root = Fr(math.isqrt(ms.numerator), math.isqrt(ms.denominator))
        assert root * root == ms
        lam_t = lam0 / root
        w = eq10_exact(w, wb, g, eta, lam_t)
        assert (float(ms), float(lam_t), float(w)) == (p["ms"], p["lambda_t"], p["w"])
    for dt in (np.float32, np.float64):
        s = oracle.Server([ex["w_bak"]], 1, True, ex["eta"], ex["lambda0"], ex["mu"], ex["eps"],
                          dtype=dt, library=L)
        assert s.ms[0] == 0.0                                     # MeanSquare(0) = 0
        s.w[0] = ex["w0"]
        for p in ex["pushes"]:
            s.push(0, np.asarray([p["g"]], dtype=dt))
            assert float(s.ms[0]) == p["ms"]
            assert float(s.w[0]) == p["w"]


def pin_exact_rational_replay(L):
    """Random small logs with dyadic inputs: the binary64 checker must equal Algorithm 2 over
    the rationals exactly (no rounding occurs), for w and for every backup."""
    rng = np.random.default_rng(11)
    for trial in range(12):
        n, M, P = 5, 3, 8
        w0 = rng.integers(-32, 33, n) / 16.0
        grads = rng.choice([-1.0, -0.5, 0.5, 1.0], size=(P, n))
        recs = [(PULL, m) for m in range(M) if rng.random() < 0.5]
        for e in range(P):
            m = int(rng.integers(M))
            recs.append((PUSH, m, e, 0.5 if e % 3 else 0.25))
            if rng.random() < 0.7:
                recs.append((PULL, int(rng.integers(M))))
        ev = synth.make_log(recs)
        eta, lam = 0.5, [0.5, 1.0, 2.0][trial % 3]
        s = oracle.Server(w0, M, False, eta, lam, dtype=np.float64, library=L)
        s.replay(ev, np.ascontiguousarray(grads, dtype=np.float64))
        w_ex, wb_ex = replay_exact(w0, M, ev, grads, Fr(eta), Fr(lam))
        assert [Fr(float(x)) for x in s.w] == w_ex
        for m in range(M):
            assert [Fr(float(x)) for x in s.w_bak[m]] == wb_ex[m]
        assert s.step == P


def _random_case(seed, n=257, M=4, pushes=60, proto=synth.PROTO_ASYNC, G=7, bf16=False):
    ev = synth.event_log(M, pushes, synth.ORDER_UNIFORM, proto, G, eta=0.1, seed=seed)
    w0 = synth.normal(n, seed, synth.STREAM_W0, 0.05)
    grads = np.stack([synth.normal(n, seed, synth.STREAM_GRAD0 + k, 0.01, bf16=bf16) for k in range(G)])
    return ev, w0, grads


def _widen(g):
    if g.dtype == np.uint16:
        return (g.astype(np.uint32) << 16).view(np.float32)
    return g


def pin_lambda0_is_asgd(L):
    """lambda = 0 turns DC-ASGD into ASGD, w <- w - eta*g (Section 2's ASGD rule; Section 5)."""
    for adaptive in (False, True):
        for bf16 in (False, True):
            ev, w0, grads = _random_case(3, bf16=bf16)
            s = oracle.Server(w0, 4, adaptive, 0.1, 0.0, 0.95, 1e-7, library=L)
            s.replay(ev, grads)
            w = w0.copy()
            for r in ev[ev["kind"] == PUSH]:
                w = w - np.float32(r["eta"]) * _widen(grads[r["grad_id"]])
            assert np.array_equal(s.w, w)


def pin_tau0_is_sgd(L):
    """A pull right before every push makes w - w_bak(m) vanish: sequential SGD, both variants."""
    for adaptive, lam in ((False, 0.04), (True, 2.0)):
        ev, w0, grads = _random_case(4, proto=synth.PROTO_TAU0)
        assert np.all(synth.delays(ev, 4) == 0)
        s = oracle.Server(w0, 4, adaptive, 0.1, lam, 0.95, 1e-7, library=L)
        s.replay(ev, grads)
        w = w0.copy()
        for r in ev[ev["kind"] == PUSH]:
            w = w - np.float32(r["eta"]) * grads[r["grad_id"]]
        assert np.array_equal(s.w, w)
        # and with real delays the compensation does change the result
        ev2, _, _ = _random_case(4, proto=synth.PROTO_ASYNC)
        s2 = oracle.Server(w0, 4, adaptive, 0.1, lam, 0.95, 1e-7, library=L)
        s2.replay(ev2, grads)
        assert not np.array_equal(s2.w, w)


def pin_meansquare_unrolled(L):
    """MeanSquare(T) = (1-mu) * sum_k mu^(T-k) g_k^2 (the recurrence of Section 6, unrolled,
    MeanSquare(0)=0); mu = 0 gives g^2 (the paper's ImageNet setting)."""
    ev, w0, grads = _random_case(6, n=64, pushes=50, G=50)
    mu = 0.95
    order = [int(r["grad_id"]) for r in ev[ev["kind"] == PUSH]]
    T = len(order)
    g64 = grads.astype(np.float64)
    want = (1 - mu) * sum(mu ** (T - 1 - k) * g64[order[k]] ** 2 for k in range(T))
    s64 = oracle.Server(w0.astype(np.float64), 4, True, 0.1, 2.0, mu, 1e-7, dtype=np.float64, library=L)
    s64.replay(ev, g64)
    assert np.allclose(s64.ms, want, rtol=1e-12, atol=0)
    s32 = oracle.Server(w0, 4, True, 0.1, 2.0, np.float32(mu), 1e-7, library=L)
    s32.replay(ev, grads)
    assert np.allclose(s32.ms, want, rtol=2e-5, atol=0)
    s0 = oracle.Server(w0, 4, True, 0.1, 2.0, 0.0, 1e-7, library=L)
    s0.replay(ev, grads)
    assert np.array_equal(s0.ms, grads[order[-1]] * grads[order[-1]])


def pin_adaptive_lambda_definition(L):
    """lambda_t = lambda_0 / sqrt(MeanSquare(t) + eps), eps inside the root, MeanSquare already
    holding the current gradient: one push from MeanSquare(0)=0 in binary64."""
    rng = np.random.default_rng(9)
    n = 16
    w0, wb, g = rng.normal(size=n), rng.normal(size=n), rng.normal(size=n) * 1e-3
    mu, lam0, eps, eta = 0.9, 2.0, 1e-7, 0.1
    s = oracle.Server(wb, 1, True, eta, lam0, mu, eps, dtype=np.float64, library=L)
    s.w[:] = w0
    s.push(0, g)
    ms = (1 - mu) * g * g
    lam = lam0 / np.sqrt(ms + eps)
    want = w0 - eta * (g + lam * g * g * (w0 - wb))
    assert np.allclose(s.w, want, rtol=1e-13, atol=1e-15)
    # eps matters at this gradient scale: outside the root the result would differ visibly
    wrong = w0 - eta * (g + (lam0 / (np.sqrt(ms) + eps)) * g * g * (w0 - wb))
    assert not np.allclose(wrong, want, rtol=1e-6, atol=0)


def pin_protocol(L):
    """Initialize sets every backup to w_0 (a push with no pull is measured against w_0); a
    pull copies only that worker's backup; only pushes advance t; the right worker's backup
    and the right gradient buffer are used."""
    w0 = np.asarray([1.0, -2.0, 0.5], dtype=np.float64)
    g = np.asarray([[0.5, 0.25, -1.0], [1.0, 1.0, 1.0], [-0.5, 0.5, 0.25]], dtype=np.float64)
    ev = synth.make_log([(PUSH, 0, 1, 0.5), (PULL, 1), (PUSH, 0, 2, 0.25), (PUSH, 1, 0, 0.5), (PULL, 0)])
    s = oracle.Server(w0, 2, False, 0.5, 2.0, dtype=np.float64, library=L)
    assert np.array_equal(s.w_bak[0], w0) and np.array_equal(s.w_bak[1], w0) and s.step == 0
    s.replay(ev, g)
    w_ex, wb_ex = replay_exact(w0, 2, ev, g, Fr(1, 2), Fr(2))
    assert [Fr(float(x)) for x in s.w] == w_ex
    assert [[Fr(float(x)) for x in s.w_bak[m]] for m in range(2)] == wb_ex
    assert s.step == 3
    assert np.array_equal(s.w_bak[0], s.w) and not np.array_equal(s.w_bak[1], s.w)


def pin_bruteforce_f32(L):
    """Element-outer scalar replay in numpy binary32 on tiny inputs, bit for bit (the same
    rounding order the checker documents), both variants, fp32 and bf16 gradients."""
    f = np.float32
    for adaptive in (False, True):
        for bf16 in (False, True):
            ev, w0, grads = _random_case(8, n=7, M=3, pushes=25, G=5, bf16=bf16)
            eta, lam, mu, eps = f(0.1), f(2.0 if adaptive else 0.04), f(0.95), f(1e-7)
            s = oracle.Server(w0, 3, adaptive, eta, lam, mu, eps, library=L)
            s.replay(ev, grads)
            gw = _widen(grads)
            for i in range(7):
                w, ms, wb = f(w0[i]), f(0), [f(w0[i])] * 3
                for r in ev:
                    m = int(r["worker"])
                    if r["kind"] == PULL:
                        wb[m] = w
                        continue
                    g = f(gw[r["grad_id"], i])
                    gg = f(g * g)
                    l = lam
                    if adaptive:
                        ms = f(f(mu * ms) + f(f(f(1) - mu) * gg))
                        l = f(lam / np.sqrt(f(ms + eps), dtype=f))
                    c = f(f(l * gg) * f(w - wb[m]))
                    w = f(w - f(f(r["eta"]) * f(g + c)))
                assert w == s.w[i] and all(wb[m] == s.w_bak[m, i] for m in range(3))
                if adaptive:
                    assert ms == s.ms[i]


def pin_f32_tracks_f64(L):
    """On a workload-shaped trajectory the binary32 replay stays within the parity tolerance
    1e-5*(1+|w|) of the binary64 replay: rounding does not amplify along the log."""
    for adaptive, lam in ((False, 0.04), (True, 2.0)):
        ev, w0, grads = _random_case(12, n=512, M=8, pushes=2000, G=64)
        s32 = oracle.Server(w0, 8, adaptive, 0.1, lam, 0.95, 1e-7, library=L)
        s64 = oracle.Server(w0.astype(np.float64), 8, adaptive, 0.1, lam, 0.95, 1e-7, dtype=np.float64, library=L)
        s32.replay(ev, grads)
        s64.replay(ev, grads.astype(np.float64))
        assert np.all(np.abs(s32.w - s64.w) <= 1e-5 * (1 + np.abs(s64.w)))


def pin_delay_compensated_ssgd(L):
    """Supplementary, "Large mini-batch synchronous SGD with delay-compensated gradient": M
    gradients all computed at w_t are applied one after another with eta_hat/M, each compensated
    against the shared snapshot w_t.  Expressed as a log (all workers pull, then all push), the
    checker must equal that recursion over the rationals; with lambda = 0 it is the plain
    large-batch step w_t - eta_hat * mean(g)."""
    rng = np.random.default_rng(21)
    n, M, rounds = 4, 4, 2
    eta_hat, lam = Fr(1, 2), Fr(2)
    w0 = rng.integers(-16, 17, n) / 8.0
    grads = rng.choice([-1.0, -0.5, 0.5, 1.0], size=(M * rounds, n))
    ev = synth.event_log(M, M * rounds, synth.ORDER_UNIFORM, synth.PROTO_SYNC, M * rounds, float(eta_hat / M), seed=4)
    for lam_ in (lam, Fr(0)):
        s = oracle.Server(w0, M, False, float(eta_hat / M), float(lam_), dtype=np.float64, library=L)
        s.replay(ev, np.ascontiguousarray(grads, dtype=np.float64))
        w = [Fr(x) for x in w0]
        pushes = ev[ev["kind"] == PUSH]
        for r in range(rounds):
            wt = list(w)                                  # the snapshot every worker pulled
            gsum = [Fr(0)] * n
            for rec in pushes[r * M:(r + 1) * M]:
                g = [Fr(float(x)) for x in grads[int(rec["grad_id"])]]
                w = [w[i] - eta_hat / M * (g[i] + lam_ * g[i] * g[i] * (w[i] - wt[i])) for i in range(n)]
                gsum = [a + b for a, b in zip(gsum, g)]
            if lam_ == 0:
                assert w == [wt[i] - eta_hat * gsum[i] / M for i in range(n)]
        assert [Fr(float(x)) for x in s.w] == w


def pin_momentum(L):
    """Momentum reading v = beta*v + eta*u ; w = w - v (u = the delay-compensated gradient):
    beta = 0 is the plain update bit for bit; with lambda = 0 and no delay it is textbook
    heavy-ball SGD (independent numpy loop, bit for bit); with dyadic inputs the binary64
    checker equals the recursion over the rationals exactly; the velocity starts at 0 and a
    pull does not touch it."""
    f = np.float32
    for adaptive, lam in ((False, 0.04), (True, 2.0)):
        ev, w0, grads = _random_case(31, n=130, pushes=40)
        plain = oracle.Server(w0, 4, adaptive, 0.1, lam, 0.95, 1e-7, library=L)
        zero = oracle.Server(w0, 4, adaptive, 0.1, lam, 0.95, 1e-7, library=L, beta=0.0)
        some = oracle.Server(w0, 4, adaptive, 0.1, lam, 0.95, 1e-7, library=L, beta=0.9)
        for s in (plain, zero, some):
            s.replay(ev, grads)
        assert np.array_equal(plain.w, zero.w) and np.array_equal(plain.w_bak, zero.w_bak)
        assert not np.array_equal(plain.w, some.w)
    # textbook momentum SGD: lambda = 0, pull right before every push
    ev, w0, grads = _random_case(32, proto=synth.PROTO_TAU0)
    s = oracle.Server(w0, 4, False, 0.1, 0.0, library=L, beta=f(0.9))
    assert np.all(s.v == 0)
    s.replay(ev, grads)
    w, v = w0.copy(), np.zeros_like(w0)
    for r in ev[ev["kind"] == PUSH]:
        v = f(0.9) * v + f(r["eta"]) * grads[r["grad_id"]]
        w = w - v
    assert np.array_equal(s.w, w) and np.array_equal(s.v, v)
    # exact rational recursion with delays and compensation, dyadic inputs, binary64
    rng = np.random.default_rng(33)
    n, M, P = 4, 3, 6
    w0 = rng.integers(-16, 17, n) / 8.0
    g = rng.choice([-1.0, -0.5, 0.5, 1.0], size=(P, n))
    recs = []
    for e in range(P):
        recs += [(PUSH, int(rng.integers(M)), e, 0.5), (PULL, int(rng.integers(M)))]
    ev = synth.make_log(recs)
    beta, eta, lam = Fr(1, 2), Fr(1, 2), Fr(1)
    s = oracle.Server(w0, M, False, float(eta), float(lam), dtype=np.float64, library=L, beta=float(beta))
    s.replay(ev, np.ascontiguousarray(g))
    w = [Fr(x) for x in w0]
    wb = [list(w) for _ in range(M)]
    v = [Fr(0)] * n
    for r in ev:
        m = int(r["worker"])
        if r["kind"] == PULL:
            wb[m] = list(w)
            continue
        gi = [Fr(float(x)) for x in g[int(r["grad_id"])]]
        u = [gi[i] + lam * gi[i] * gi[i] * (w[i] - wb[m][i]) for i in range(n)]
        v = [beta * v[i] + eta * u[i] for i in range(n)]
        w = [w[i] - v[i] for i in range(n)]
    assert [Fr(float(x)) for x in s.w] == w and [Fr(float(x)) for x in s.v] == v


PINS = [pin_hand_constant, pin_closed_form_repeated, pin_hand_adaptive, pin_exact_rational_replay,
        pin_lambda0_is_asgd, pin_tau0_is_sgd, pin_meansquare_unrolled, pin_adaptive_lambda_definition,
        pin_protocol, pin_bruteforce_f32, pin_f32_tracks_f64, pin_delay_compensated_ssgd, pin_momentum]


@pytest.mark.parametrize("pin", PINS, ids=lambda p: p.__name__)
def test_pin(pin, oracle_lib):
    pin(oracle_lib)


def test_replay_rejects_bad_records(oracle_lib):
    w0 = np.zeros(4, dtype=np.float32)
    g = np.zeros((2, 4), dtype=np.float32)
    for recs in ([(PUSH, 5, 0)], [(PUSH, 0, 2)], [(7, 0, 0)]):
        s = oracle.Server(w0, 2, False, 0.1, 0.04)
        with pytest.raises(ValueError):
            s.replay(synth.make_log(recs), g)
