"""Algorithmic HBM bytes of the server's operations (what the method must move, per element)
and multi-rank aggregation of timings.  Host-side bookkeeping only; no arithmetic of the update.

Per element, fp32 state:
    pull                      8            read w, write w_bak[m]
    push, constant lambda    12 + g        w in and out, w_bak[m] in, gradient in (g = 4 fp32, 2 bf16)
    push, adaptive           20 + g        + MeanSquare in and out
    (momentum variant: + 8 per push, or per window, for the velocity in and out)
    fused window              S + g*P + 4*R + 4*W
        S = 8 (constant) or 16 (adaptive): w (and ms) in and out once per window
        P = pushes in the window, R = pushes that read a pre-window backup,
        W = backups written (the last pull of each worker in the window)
"""
from __future__ import annotations


def grad_bytes(bf16: bool) -> int:
    return 2 if bf16 else 4


def pull_bytes() -> int:
    return 8


def push_bytes(adaptive: bool, bf16: bool, momentum: bool = False) -> int:
    return (20 if adaptive else 12) + grad_bytes(bf16) + (8 if momentum else 0)


def init_bytes(M: int, adaptive: bool) -> int:
    return 4 + 4 * M + (4 if adaptive else 0)


def window_bytes(prog, adaptive: bool, bf16: bool, momentum: bool = False) -> int:
    """Bytes per element of one compiled window (a WindowProgram); 0 if it launches nothing."""
    if prog.n_pushes == 0 and prog.n_stores == 0:
        return 0
    state = (16 if adaptive else 8) + (8 if momentum else 0)
    return state + grad_bytes(bf16) * prog.n_pushes + 4 * prog.n_snapshot_reads + 4 * prog.n_stores


def unfused_log_bytes(n_pushes: int, n_pulls: int, adaptive: bool, bf16: bool) -> int:
    return n_pushes * push_bytes(adaptive, bf16) + n_pulls * pull_bytes()


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None) -> tuple[float, float]:
    """Whole-job view of a timed region run by independent replicas: the time is the slowest
    rank's, the units are summed.  `dist` is torch.distributed (initialised) or None for one
    process.  Returns (max_ms, total_units)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
