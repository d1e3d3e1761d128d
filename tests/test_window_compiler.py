"""Host logic of the fused replay (no GPU): the window compiler's step programs, interpreted on
the CPU with the checker's own push for the arithmetic, must reproduce the checker's serial
replay bit for bit - for random logs, every window size, and logs built to hit the slot,
push and store limits."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth

PULL, PUSH = B.PULL, B.PUSH


def interpret(programs, w0, M, adaptive, lam, mu, eps, grads):
    """Runs step programs the way the kernel does for one element block, on the host."""
    n = w0.size
    w = w0.copy()
    w_bak = np.tile(w0, (M, 1))
    one = oracle.Server(w0, 1, adaptive, 0.0, lam, mu, eps)      # arithmetic engine: one push at a time
    one.w[:] = w0
    for p in programs:
        slots, stored = {}, set()

        def after(j):
            if p.save_slot[j] >= 0:
                slots[p.save_slot[j]] = one.w.copy()
            for k in range(p.store_begin[j], p.store_begin[j + 1]):
                w_bak[p.store_worker[k]] = one.w
                stored.add(p.store_worker[k])
        pre = w_bak.copy()                    # pre-window backups are what src >= 0 refers to
        after(0)
        for j in range(p.n_pushes):
            src = p.src[j]
            snap = pre[src] if src >= 0 else slots[-(src + 1)]
            # the kernel may read a pre-window backup early: nothing in this window may have
            # written that slab before the push that uses it
            assert src < 0 or src not in stored
            one.w_bak[0] = snap
            one.push(0, grads[p.grad_id[j]], float(p.eta[j]))
            after(j + 1)
        assert len(slots) <= B.MAX_WINDOW_SLOTS
    return one.w.copy(), w_bak, (one.ms.copy() if adaptive else None)


def serial(ev, w0, M, adaptive, eta, lam, mu, eps, grads):
    s = oracle.Server(w0, M, adaptive, eta, lam, mu, eps)
    s.replay(ev, grads)
    return s


def check(ev, M, K, adaptive=True, n=9, G=5, seed=0, eta=0.1, max_slots=0):
    w0 = synth.normal(n, seed, synth.STREAM_W0, 0.05)
    grads = np.stack([synth.normal(n, seed, synth.STREAM_GRAD0 + k, 0.01) for k in range(G)])
    lam, mu, eps = (2.0, 0.95, 1e-7) if adaptive else (0.04, 0.0, 0.0)
    progs = B.plan_log(ev, M, K, eta, max_slots)
    assert sum(p.n_records for p in progs) == len(ev)
    assert sum(p.n_pushes for p in progs) == int(np.sum(ev["kind"] == PUSH))
    w, wb, ms = interpret(progs, w0, M, adaptive, lam, mu, eps, grads)
    ref = serial(ev, w0, M, adaptive, eta, lam, mu, eps, grads)
    assert np.array_equal(w, ref.w)
    assert np.array_equal(wb, ref.w_bak)
    if adaptive:
        assert np.array_equal(ms, ref.ms)
    return progs


@pytest.mark.parametrize("K", [2, 3, 8, 32, 64, 257, 1000])
@pytest.mark.parametrize("order,M", [(synth.ORDER_UNIFORM, 16), (synth.ORDER_ROUND_ROBIN_JITTER, 4),
                                     (synth.ORDER_ZIPF, 32), (synth.ORDER_UNIFORM, 1)])
def test_random_logs_every_window_size(K, order, M):
    ev = synth.event_log(M, 300, order, synth.PROTO_ASYNC, 5, 0.1, seed=K, order_param=1.2)
    progs = check(ev, M, K)
    for p in progs:
        assert 1 <= p.n_records <= K
        assert p.n_pushes <= B.MAX_WINDOW_PUSHES and p.n_stores <= B.MAX_WINDOW_STORES
        assert p.n_slots <= B.MAX_WINDOW_SLOTS


def test_other_protocols_and_constant_variant():
    for proto in (synth.PROTO_TAU0, synth.PROTO_SYNC):
        ev = synth.event_log(6, 120, synth.ORDER_UNIFORM, proto, 5, 0.05, seed=3)
        check(ev, 6, 16, adaptive=False)
        check(ev, 6, 7, adaptive=True)


def test_arbitrary_record_soup():
    """Not a worker loop at all: random kinds, repeated pulls, pushes without pulls, per-record eta."""
    rng = np.random.default_rng(0)
    for trial in range(30):
        M = int(rng.integers(1, 6))
        recs = []
        for _ in range(int(rng.integers(1, 80))):
            if rng.random() < 0.5:
                recs.append((PUSH, int(rng.integers(M)), int(rng.integers(5)), float(rng.choice([-1.0, 0.05, 0.2]))))
            else:
                recs.append((PULL, int(rng.integers(M))))
        check(synth.make_log(recs), M, int(rng.integers(2, 40)), adaptive=bool(trial % 2))


def test_byte_accounting_of_a_window():
    # PULL(0) PULL(1) | PUSH(0) PULL(0) PUSH(1) PULL(1) PUSH(0) PULL(0) in one window
    ev = synth.make_log([(PULL, 0), (PULL, 1), (PUSH, 0, 0), (PULL, 0), (PUSH, 1, 1), (PULL, 1), (PUSH, 0, 2), (PULL, 0)])
    (p,) = B.plan_log(ev, 2, 64, 0.1)
    assert (p.n_records, p.n_pushes) == (8, 3)
    # both first pushes use the snapshots pulled at the head of the window (the incoming w, one slot);
    # the third push uses worker 0's snapshot taken after push 0
    assert p.n_snapshot_reads == 0
    assert list(p.src[:3]) == [-(p.save_slot[0] + 1), -(p.save_slot[0] + 1), -(p.save_slot[1] + 1)]
    # only the last pull of each worker is written: worker 1 after push 1, worker 0 after push 2
    assert p.n_stores == 2 and p.n_dead_pulls == 0
    assert [list(p.store_worker[p.store_begin[j]:p.store_begin[j + 1]]) for j in range(4)] == [[], [], [1], [0]]
    # with the same records spread over windows of 2, every push reads a pre-window backup
    progs = B.plan_log(ev, 2, 2, 0.1)
    assert sum(q.n_snapshot_reads for q in progs) == 3 and sum(q.n_stores for q in progs) == 5
    # a superseded, unused pull costs nothing
    (q,) = B.plan_log(synth.make_log([(PULL, 0), (PULL, 0), (PUSH, 0, 0)]), 1, 8, 0.1)
    assert q.n_dead_pulls == 1 and q.n_stores == 1 and q.n_snapshot_reads == 0


def test_limits_cut_the_window():
    M = 40
    # more live in-window snapshots than slots: worker k pulls after push k, uses it much later
    recs = []
    for k in range(M):
        recs += [(PUSH, k, k % 5), (PULL, k)]
    for k in range(M):
        recs += [(PUSH, k, k % 5)]
    ev = synth.make_log(recs)
    progs = check(ev, M, 1000, G=5)
    assert len(progs) > 1 and max(p.n_slots for p in progs) == B.MAX_WINDOW_SLOTS
    # more pushes than a window holds
    ev = synth.make_log([(PUSH, 0, k % 5) for k in range(1500)])
    progs = check(ev, 1, 1_000_000, G=5)
    assert [p.n_pushes for p in progs] == [B.MAX_WINDOW_PUSHES, B.MAX_WINDOW_PUSHES, 1500 - 2 * B.MAX_WINDOW_PUSHES]
    # more final pulls than a window can store
    ev = synth.make_log([(PUSH, 0, 0)] + [(PULL, m) for m in range(1100)] + [(PUSH, 3, 1)])
    progs = check(ev, 1100, 1_000_000, G=5)
    assert progs[0].n_stores == B.MAX_WINDOW_STORES and len(progs) == 2


def test_compile_rejects_bad_records():
    for recs in ([(2, 0)], [(PUSH, 4, 0)], [(PUSH, 0, 0, float("nan"))]):
        with pytest.raises(B.DcasgdError) as e:
            B.dcasgd_compile_window(synth.make_log(recs), 4, 8, 0.1)
        assert e.value.status == B.ELOG
    with pytest.raises(B.DcasgdError) as e:
        B.dcasgd_compile_window(synth.make_log([]), 4, 8, 0.1)
    assert e.value.status == B.EINVAL


@pytest.mark.parametrize("cap", [1, 2, 3, 8, 16])
def test_slot_cap_cuts_windows_but_not_results(cap):
    """A smaller slot budget ends windows earlier; the replay stays the checker's, bit for bit."""
    ev = synth.event_log(16, 400, synth.ORDER_UNIFORM, synth.PROTO_ASYNC, 5, 0.1, seed=cap)
    progs = check(ev, 16, 256, max_slots=cap)
    assert max(p.n_slots for p in progs) <= cap
    full = B.plan_log(ev, 16, 256, 0.1)
    assert len(progs) >= len(full)
    if cap == 16:
        assert [p.n_records for p in progs] == [p.n_records for p in full]
    with pytest.raises(B.DcasgdError):
        B.dcasgd_compile_window(ev, 16, 8, 0.1, max_slots=17)


def test_huge_window_k_stays_linear_in_the_log():
    """window_k far beyond what a window can hold: the compiler bounds the records it scans per
    window, so planning a long log takes time proportional to the log (and cuts it correctly)."""
    import time
    ev = synth.event_log(16, 60_000, synth.ORDER_UNIFORM, synth.PROTO_ASYNC, 5, 0.1, seed=11)
    t0 = time.perf_counter()
    progs = B.plan_log(ev, 16, 2 ** 32 - 1, 0.1)
    dt = time.perf_counter() - t0
    assert sum(p.n_records for p in progs) == len(ev)
    assert all(p.n_records <= 2048 for p in progs)
    assert dt < 20.0, f"planning {len(ev)} records took {dt:.1f} s"
    check(ev[:3000], 16, 2 ** 32 - 1)
