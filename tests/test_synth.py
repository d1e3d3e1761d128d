"""Properties of the seeded input generator (no GPU)."""
import numpy as np
import pytest

from paper_1609_08326_b200 import synth

PULL, PUSH = synth.PULL, synth.PUSH


def test_event_record_layout():
    assert synth.EVENT_DTYPE.itemsize == 16
    ev = synth.make_log([(PUSH, 3, 7, 0.25)])
    raw = ev.view(np.uint8)
    assert raw[0] == 1 and raw[4] == 3 and raw[8] == 7
    assert np.frombuffer(raw[12:16].tobytes(), dtype=np.float32)[0] == 0.25


def test_values_are_a_function_of_seed_stream_index():
    a = synth.normal(10_001, 7, 5, 0.5)
    assert np.array_equal(a, synth.normal(10_001, 7, 5, 0.5, threads=1))
    assert np.array_equal(a[1234:2001], synth.normal(767, 7, 5, 0.5, first=1234))
    idx = [0, 3, 4, 9_999, 10_000]
    assert np.array_equal(a[idx], synth.normal_gather(idx, 7, 5, 0.5))
    assert not np.array_equal(a, synth.normal(10_001, 8, 5, 0.5))
    assert not np.array_equal(a, synth.normal(10_001, 7, 6, 0.5))
    big = synth.normal(300_000, 1, 2, 1.0)            # threaded path
    assert np.array_equal(big, synth.normal(300_000, 1, 2, 1.0, threads=1))


def test_normal_moments_and_segments():
    z = synth.normal(400_000, 0, 9, 1.0)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    assert abs(np.mean(z ** 4) - 3) < 0.1
    sig = synth.log_uniform_sigma(60, -4, -1, 0)
    assert np.all((sig >= 1e-4) & (sig <= 1e-1))
    n, nseg = 100_003, 7
    s7 = sig[:nseg]
    x = synth.normal(n, 0, 9, s7, seg_len=n // nseg)
    assert np.array_equal(x[: n // nseg], (z[: n // nseg] * s7[0]).astype(np.float32))
    assert np.array_equal(x[-3:], (z[n - 3:n] * s7[-1]).astype(np.float32))    # remainder: last segment


def test_bf16_is_round_to_nearest_even_of_the_f32_values():
    f = synth.normal(4096, 3, 11, 0.01)
    h = synth.normal(4096, 3, 11, 0.01, bf16=True)
    u = f.view(np.uint32).astype(np.uint64)
    want = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    assert np.array_equal(h, want)
    wide = (h.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(wide[[1, 77]], synth.normal_gather([1, 77], 3, 11, 0.01, through_bf16=True))
    assert np.all(np.abs(wide - f) <= np.abs(f) * 2.0 ** -8)


@pytest.mark.parametrize("order,param", [(synth.ORDER_ROUND_ROBIN_JITTER, 0), (synth.ORDER_UNIFORM, 0),
                                         (synth.ORDER_ZIPF, 1.2)])
def test_async_log_follows_the_worker_loop(order, param):
    M, P, G = 8, 3000, 64
    ev = synth.event_log(M, P, order, synth.PROTO_ASYNC, G, 0.1, seed=1, order_param=param)
    assert np.array_equal(ev, synth.event_log(M, P, order, synth.PROTO_ASYNC, G, 0.1, seed=1, order_param=param))
    assert len(ev) == M + 2 * P
    assert np.all(ev["kind"][:M] == PULL) and np.array_equal(ev["worker"][:M], np.arange(M))
    body = ev[M:]
    assert np.all(body["kind"][0::2] == PUSH) and np.all(body["kind"][1::2] == PULL)
    assert np.array_equal(body["worker"][0::2], body["worker"][1::2])      # pull right after own push
    assert np.array_equal(body["grad_id"][0::2], np.arange(P) % G)
    assert np.all(ev["worker"] < M) and np.all(ev["eta"] == np.float32(0.1))


def test_delay_statistics():
    # uniform pusher: geometric delay with mean M-1
    d = synth.delays(synth.event_log(8, 20000, synth.ORDER_UNIFORM, seed=0), 8)
    assert abs(d.mean() - 7) < 0.3
    # round robin with +-1 jitter: delay stays near M-1
    ev = synth.event_log(4, 2000, synth.ORDER_ROUND_ROBIN_JITTER, seed=0)
    d = synth.delays(ev, 4)
    assert abs(d.mean() - 3) < 0.1 and d.max() <= 6
    assert np.bincount(ev["worker"][ev["kind"] == PUSH], minlength=4).tolist() == [500] * 4
    # Zipf speeds: slow workers see far longer delays than fast ones
    ev = synth.event_log(32, 2000, synth.ORDER_ZIPF, seed=0, order_param=1.2)
    d = synth.delays(ev, 32)
    who = ev["worker"][ev["kind"] == PUSH]
    assert d[who == 0].mean() < 4 and d[who >= 24].mean() > 100
    # tau = 0 protocol
    assert np.all(synth.delays(synth.event_log(4, 100, synth.ORDER_UNIFORM, synth.PROTO_TAU0), 4) == 0)


def test_sync_rounds():
    M = 4
    ev = synth.event_log(M, 10, synth.ORDER_UNIFORM, synth.PROTO_SYNC, 3, seed=2)
    assert len(ev) == 2 * 2 * M                      # 10 pushes -> 2 whole rounds
    for r in range(2):
        blk = ev[r * 2 * M:(r + 1) * 2 * M]
        assert np.all(blk["kind"][:M] == PULL) and np.all(blk["kind"][M:] == PUSH)
        assert sorted(blk["worker"][M:].tolist()) == list(range(M))


def test_workload_recipes():
    names = synth.workload_names()
    assert names[:3] == ["c1_resnet20_const", "c2_adaptive_1p7m", "c3_resnet50_adaptive"]
    w = synth.workload("c3_resnet50_adaptive")
    assert (w.n, w.M, w.pushes, w.nseg) == (25_557_032, 16, 5_000, 161)
    small = w.scaled(n=1000, pushes=10, num_grads=4)
    assert small.grad(1).shape == (1000,) and np.array_equal(small.grad(1)[[5, 999]], small.grad(1, idx=[5, 999]))
    assert len(small.log()) == 16 + 20
