"""Helpers shared by the GPU parity tests: build inputs once on the host, hand the same bytes
to the CUDA library (through the C ABI) and to the CPU checker, compare element by element."""
from __future__ import annotations

import numpy as np

import oracle
from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth


def row_elems(n: int) -> int:
    return (n + 31) // 32 * 32


def host_pool(wl: synth.Workload, G: int | None = None) -> np.ndarray:
    """[G][row] gradient pool on the host (float32 values or uint16 bfloat16 patterns); row padded
    to 32 elements so that every buffer starts 16-byte aligned."""
    G = G or wl.num_grads
    pool = np.zeros((G, row_elems(wl.n)), dtype=np.uint16 if wl.bf16_grad else np.float32)
    for k in range(G):
        wl.grad_into(pool[k, : wl.n], k)
    return pool


def to_device(pool: np.ndarray):
    import torch
    if pool.dtype == np.uint16:
        return torch.from_numpy(pool.view(np.int16)).cuda()
    return torch.from_numpy(pool).cuda()


def gpu_server(wl: synth.Workload, w0: np.ndarray, stream=None, beta=None) -> B.Server:
    return B.Server(w0, wl.M, wl.adaptive, wl.eta, wl.lam, wl.mu, wl.eps, wl.bf16_grad, stream=stream, beta=beta)


def cpu_server(wl: synth.Workload, w0: np.ndarray, beta=None) -> oracle.Server:
    return oracle.Server(w0, wl.M, wl.adaptive, np.float32(wl.eta), np.float32(wl.lam), np.float32(wl.mu),
                         np.float32(wl.eps), beta=None if beta is None else np.float32(beta))


def sample_indices(n: int, seg_len: int = 0, nseg: int = 1, edge: int = 4096, every: int = 1009) -> np.ndarray:
    """Head and tail of the vector, +-8 around every segment boundary, and a regular stride."""
    parts = [np.arange(min(edge, n)), np.arange(max(0, n - edge), n), np.arange(0, n, every)]
    if seg_len:
        for s in range(1, nseg):
            b = s * seg_len
            parts.append(np.arange(max(0, b - 8), min(n, b + 8)))
    return np.unique(np.concatenate(parts)).astype(np.int64)


def assert_state_equal(gpu: B.Server, cpu: oracle.Server, idx: np.ndarray | None = None, what: str = "") -> None:
    """Bit-for-bit comparison of w, every w_bak slab and ms (all of them, or the sampled
    elements `idx` when the checker ran on a subset); also the stated tolerance, spelled out."""
    import torch
    torch.cuda.synchronize()
    sel = (lambda t: t.cpu().numpy()) if idx is None else (lambda t: t[..., torch.from_numpy(idx).cuda()].cpu().numpy())
    pairs = [("w", sel(gpu.w), cpu.w), ("w_bak", sel(gpu.w_bak), cpu.w_bak)]
    if cpu.ms is not None:
        pairs.append(("ms", sel(gpu.ms), cpu.ms))
    if cpu.v is not None:
        pairs.append(("v", sel(gpu.v), cpu.v))
    for name, got, want in pairs:
        assert got.shape == want.shape
        # NaN payloads are not fixed by IEEE 754 (x86 and the GPU pick different quiet NaNs)
        same = (got.view(np.uint32) == want.view(np.uint32)) | (np.isnan(got) & np.isnan(want))
        with np.errstate(all="ignore"):
            tol_ok = np.abs(got.astype(np.float64) - want) <= 1e-5 * (1 + np.abs(want))  # max|dw| <= 1e-5 (1+|w|)
        assert np.all(tol_ok | same), f"{what}{name}: outside tolerance"
        assert np.all(same), f"{what}{name}: {np.count_nonzero(~same)} of {same.size} elements differ in bits"
    assert gpu.step == cpu.step


def cpu_replay_ranges(wl: synth.Workload, ev: np.ndarray, w0: np.ndarray, pool: np.ndarray, threads: int):
    """The checker's serial replay over the full vector, its unchanged replay function called on
    disjoint element ranges from several host threads (elements never interact).  Returns the
    per-range servers and their bounds."""
    import threading
    bounds = np.linspace(0, wl.n, threads + 1).astype(np.int64)
    servers = [cpu_server(wl, w0[lo:hi]) for lo, hi in zip(bounds[:-1], bounds[1:])]
    ths = [threading.Thread(target=s.replay, args=(ev, pool[:, lo:hi]))
           for s, lo, hi in zip(servers, bounds[:-1], bounds[1:])]
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    return servers, bounds


def assert_ranges_equal(gpu: B.Server, servers, bounds) -> None:
    import torch
    torch.cuda.synchronize()
    for s, lo, hi in zip(servers, bounds[:-1], bounds[1:]):
        pairs = [("w", gpu.w[lo:hi], s.w), ("w_bak", gpu.w_bak[:, lo:hi], s.w_bak)]
        if s.ms is not None:
            pairs.append(("ms", gpu.ms[lo:hi], s.ms))
        for name, got, want in pairs:
            got = got.cpu().numpy()
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), f"{name}[{lo}:{hi}] differs"
        assert gpu.step == s.step
