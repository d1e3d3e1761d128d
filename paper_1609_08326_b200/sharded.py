"""Element-range sharded parameter server: one rank per GPU, each owning a contiguous range of
the model and running the unchanged single-GPU server library on it.

The paper keeps one logical server but notes (Section 4, closing discussion of Algorithm 2) that
in practice it is implemented in a distributed manner.  The update rule (Section 4, Eq. 10) and
the MeanSquare rule (Section 6) are elementwise, so a rank that owns elements [lo, hi) of
w, w_bak[.], ms and v can apply every message to its range without talking to anyone:

    push(m, g)     rank r applies Algorithm 2's gradient branch to g[lo_r:hi_r]      no collective
    pull(m)        rank r copies w[lo_r:hi_r] to its w_bak[m]                         no collective
    model to the worker ("send w_t to worker m")   all-gather of the shards           NCCL
    a full gradient that sits on one rank          scatter of its slices              NCCL

Collectives are plain `torch.distributed` calls on buffers in the calling rank's own memory: no
kernel of the library is ever handed another GPU's memory.

Layout: with `chunk = ceil(n / world)` rounded up to 32 elements, rank r owns
[min(r*chunk, n), min((r+1)*chunk, n)).  Every shard therefore starts on a 128-byte boundary of
the full vector, all shards but the last have exactly `chunk` elements, and the concatenation
of the shards padded to `chunk` is the full vector followed by padding: an all-gather into a
`world*chunk` buffer reassembles the model in place.
"""
from __future__ import annotations

import numpy as np

ALIGN = 32          # elements: shard boundaries are multiples of 32 floats (128 bytes)


def chunk_elems(n: int, world: int) -> int:
    """Elements per shard (all but possibly the last ones): ceil(n / world) rounded up to ALIGN."""
    if world < 1:
        raise ValueError("world must be >= 1")
    per = -(-n // world)
    return max(ALIGN, -(-per // ALIGN) * ALIGN)


def shard_range(n: int, world: int, rank: int) -> tuple[int, int]:
    """[lo, hi) of the elements rank `rank` owns.  Trailing ranks may own nothing when n is small."""
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside [0, {world})")
    c = chunk_elems(n, world)
    return min(rank * c, n), min((rank + 1) * c, n)


def partition(n: int, world: int) -> list[tuple[int, int]]:
    return [shard_range(n, world, r) for r in range(world)]


def gather_model(local, n: int, world: int, dist=None, group=None, out=None):
    """All-gather of the shards into the full model (what a pulling worker receives).

    `local`: this rank's shard, a 1-D torch tensor of hi-lo elements (CPU with gloo, CUDA with
    NCCL).  Returns a tensor of n elements (a view of the `world*chunk` gather buffer `out`,
    allocated here when not given).  With `dist` None (one process) the shard is the model."""
    import torch
    c = chunk_elems(n, world)
    if out is None:
        out = torch.empty(world * c, dtype=local.dtype, device=local.device)
    if out.numel() != world * c:
        raise ValueError("gather buffer must hold world * chunk elements")
    if dist is None or world == 1:
        out[: local.numel()].copy_(local)
        return out[:n]
    send = local
    if local.numel() != c:                               # the last (short or empty) shard: pad to the common size
        send = torch.zeros(c, dtype=local.dtype, device=local.device)
        send[: local.numel()].copy_(local)
    dist.all_gather_into_tensor(out, send.contiguous(), group=group)
    return out[:n]


def scatter_gradient(full, n: int, world: int, rank: int, src: int, dist=None, group=None, out=None):
    """A gradient of n elements held by rank `src` is cut into the shards' slices and each slice
    sent to its owner.  `full` is needed on `src` only (None elsewhere).  Returns this rank's
    slice (hi-lo elements, a view of the chunk-sized receive buffer `out`)."""
    import torch
    c = chunk_elems(n, world)
    lo, hi = shard_range(n, world, rank)
    if dist is None or world == 1:
        return full[lo:hi]
    if out is None:
        if full is None:
            raise ValueError("ranks other than src must pass a receive buffer `out`")
        out = torch.empty(c, dtype=full.dtype, device=full.device)
    if out.numel() != c:
        raise ValueError("the receive buffer must hold chunk_elems(n, world) elements")
    if rank == src and (full is None or full.numel() < n):
        raise ValueError("rank src must pass the full gradient (n elements)")
    pieces = None
    if rank == src:
        padded = full
        if full.numel() != world * c:
            padded = torch.zeros(world * c, dtype=full.dtype, device=full.device)
            padded[:n].copy_(full[:n])
        pieces = list(padded.view(world, c).unbind(0))
    dist.scatter(out, pieces, src=src, group=group)
    return out[: hi - lo]


class ShardedServer:
    """One rank of the sharded server: the single-GPU server library over this rank's range.

    Every rank makes the same calls in the same order (the message order of Algorithm 2 is the
    call order, as for one GPU).  `dist` is `torch.distributed` (initialised, NCCL) or None when
    the ranks are driven one after the other by a single process (tests on one GPU)."""

    def __init__(self, w0_shard, n: int, rank: int, world: int, num_workers: int, adaptive: bool, eta: float,
                 lam: float, mu: float = 0.0, eps: float = 0.0, bf16_grad: bool = False, device="cuda",
                 stream=None, dist=None, group=None, beta: float | None = None):
        from . import binding as B
        self.n, self.rank, self.world = int(n), int(rank), int(world)
        self.lo, self.hi = shard_range(self.n, self.world, self.rank)
        self.chunk = chunk_elems(self.n, self.world)
        self.dist, self.group = dist, group
        w0_shard = np.asarray(w0_shard, dtype=np.float32) if not hasattr(w0_shard, "device") else w0_shard
        if int(w0_shard.shape[0] if hasattr(w0_shard, "shape") else len(w0_shard)) != self.hi - self.lo:
            raise ValueError(f"rank {rank} owns {self.hi - self.lo} elements, got {len(w0_shard)}")
        self.local = B.Server(w0_shard, num_workers, adaptive, eta, lam, mu, eps, bf16_grad, device=device,
                              stream=stream, beta=beta)
        self._gather_buf = None
        self._recv_buf = None

    # ---- the two messages of Algorithm 2, on this rank's range
    def push(self, m: int, g_slice, eta: float = -1.0) -> None:
        """g_slice: this rank's hi-lo elements of the gradient (device)."""
        self.local.push(m, g_slice, eta)

    def push_from(self, m: int, g_full, src: int, eta: float = -1.0) -> None:
        """The whole gradient sits on rank `src`: scatter its slices, then push."""
        import torch
        if self._recv_buf is None:
            dt = torch.int16 if self.local.bf16_grad else torch.float32
            self._recv_buf = torch.empty(self.chunk, dtype=dt, device=self.local.device)
        g = scatter_gradient(g_full, self.n, self.world, self.rank, src, self.dist, self.group, self._recv_buf)
        self._sync_collective_to_server()
        self.local.push(m, g, eta)

    def pull(self, m: int, gather: bool = False):
        """w_bak[m] <- w on every shard; with `gather` also returns the full model (n elements) as
        the worker receives it (all-gather of the shards into this rank's memory)."""
        import torch
        self.local.pull(m)
        if not gather:
            return None
        if self._gather_buf is None:
            self._gather_buf = torch.empty(self.world * self.chunk, dtype=torch.float32, device=self.local.device)
        self._sync_server_to_collective()
        return gather_model(self.local.w, self.n, self.world, self.dist, self.group, self._gather_buf)

    def apply_log(self, ev, grad_pool_slice, window_k: int) -> None:
        """The message loop over a recorded log; grad_pool_slice is [G][row] with this rank's
        columns of every gradient buffer."""
        self.local.apply_log(ev, grad_pool_slice, window_k)

    # ---- stream ordering between the server's stream and the stream collectives run on
    def _sync_server_to_collective(self) -> None:
        import torch
        if self.local.stream is not None:
            torch.cuda.current_stream(self.local.device).wait_stream(self.local.stream)

    def _sync_collective_to_server(self) -> None:
        import torch
        if self.local.stream is not None:
            self.local.stream.wait_stream(torch.cuda.current_stream(self.local.device))

    @property
    def step(self) -> int:
        return self.local.step

    def close(self) -> None:
        self.local.close()
