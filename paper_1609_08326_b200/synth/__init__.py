"""Seeded synthetic inputs (parameter vectors, gradient pools, worker event logs).

Thin ctypes binding over ``libdcasgd_synth.so``.  The module holds none of the method's
arithmetic: it produces bytes that both the CUDA server library and the CPU checker consume.
Every value is a pure function of ``(seed, stream, element index)``.

Workload recipes (`workload(name)`) mirror the paper's experimental shapes: parameter counts
of the networks it trains, its worker counts M and its hyper-parameters (Section 6), with
synthetic gradients in place of CIFAR-10 / ImageNet.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field, replace

import numpy as np

PULL, PUSH = 0, 1
ORDER_ROUND_ROBIN_JITTER, ORDER_UNIFORM, ORDER_ZIPF = 0, 1, 2
PROTO_ASYNC, PROTO_TAU0, PROTO_SYNC = 0, 1, 2

# stream ids (which random sequence feeds what)
STREAM_W0, STREAM_LOG, STREAM_SIGMA, STREAM_GRAD0 = 1, 2, 3, 0x1000

EVENT_DTYPE = np.dtype(
    {"names": ["kind", "worker", "grad_id", "eta"],
     "formats": [np.uint8, np.uint32, np.uint32, np.float32],
     "offsets": [0, 4, 8, 12], "itemsize": 16})

_SO = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdcasgd_synth.so")
_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            from .. import build
            build.build_synth()
        L = C.CDLL(_SO)
        u64, u32, f32p = C.c_uint64, C.c_uint32, C.c_void_p
        L.synth_hardware_threads.restype = C.c_int
        L.synth_normal_f32.argtypes = [C.c_void_p, u64, u64, u64, u64, f32p, u32, u64, C.c_int]
        L.synth_normal_f32.restype = None
        L.synth_normal_bf16.argtypes = [C.c_void_p, u64, u64, u64, u64, f32p, u32, u64, C.c_int]
        L.synth_normal_bf16.restype = None
        L.synth_normal_gather.argtypes = [C.c_void_p, C.c_void_p, u64, u64, u64, f32p, u32, u64, C.c_int]
        L.synth_normal_gather.restype = None
        L.synth_log_uniform_sigma.argtypes = [C.c_void_p, u32, C.c_double, C.c_double, u64, u64]
        L.synth_log_uniform_sigma.restype = None
        L.synth_u32.argtypes = [C.c_void_p, u64, u64, u64, u64]
        L.synth_u32.restype = None
        L.synth_event_log_size.argtypes = [u32, u64, u32]
        L.synth_event_log_size.restype = u64
        L.synth_event_log.argtypes = [C.c_void_p, u64, u32, u64, u32, C.c_double, u32, u32,
                                      C.c_float, u64, u64]
        L.synth_event_log.restype = u64
        _lib = L
    return _lib


def hardware_threads() -> int:
    return int(lib().synth_hardware_threads())


def _sigma_arr(sigma) -> np.ndarray:
    s = np.atleast_1d(np.asarray(sigma, dtype=np.float32))
    return np.ascontiguousarray(s)


def normal_into(out: np.ndarray, first: int, seed: int, stream: int, sigma=1.0,
                seg_len: int = 0, threads: int = 0) -> np.ndarray:
    """Fill a contiguous 1-D float32 (values) or uint16 (bfloat16 bit patterns) array with
    elements ``first .. first+len(out)`` of the stream."""
    assert out.ndim == 1 and out.flags.c_contiguous
    s = _sigma_arr(sigma)
    t = threads or hardware_threads()
    fn = {np.dtype(np.float32): lib().synth_normal_f32,
          np.dtype(np.uint16): lib().synth_normal_bf16}[out.dtype]
    fn(out.ctypes.data, first, out.size, seed, stream, s.ctypes.data, s.size, seg_len, t)
    return out


def normal(n: int, seed: int, stream: int, sigma=1.0, seg_len: int = 0, first: int = 0,
           bf16: bool = False, threads: int = 0) -> np.ndarray:
    out = np.empty(n, dtype=np.uint16 if bf16 else np.float32)
    return normal_into(out, first, seed, stream, sigma, seg_len, threads)


def normal_gather(idx, seed: int, stream: int, sigma=1.0, seg_len: int = 0,
                  through_bf16: bool = False) -> np.ndarray:
    """Values of the scattered elements ``idx`` of a stream, as float32 (exactly what the full
    vector would hold there; with ``through_bf16`` what the bfloat16 vector widens to)."""
    ix = np.ascontiguousarray(np.asarray(idx, dtype=np.uint64))
    s = _sigma_arr(sigma)
    out = np.empty(ix.size, dtype=np.float32)
    lib().synth_normal_gather(out.ctypes.data, ix.ctypes.data, ix.size, seed, stream,
                              s.ctypes.data, s.size, seg_len, int(through_bf16))
    return out


def log_uniform_sigma(nseg: int, lo_exp: float, hi_exp: float, seed: int,
                      stream: int = STREAM_SIGMA) -> np.ndarray:
    out = np.empty(nseg, dtype=np.float32)
    lib().synth_log_uniform_sigma(out.ctypes.data, nseg, lo_exp, hi_exp, seed, stream)
    return out


def u32(n: int, seed: int, stream: int, first: int = 0) -> np.ndarray:
    out = np.empty(n, dtype=np.uint32)
    lib().synth_u32(out.ctypes.data, first, n, seed, stream)
    return out


def event_log(M: int, pushes: int, order: int, proto: int = PROTO_ASYNC, num_grads: int = 1,
              eta: float = 0.1, seed: int = 0, order_param: float = 0.0,
              stream: int = STREAM_LOG) -> np.ndarray:
    """Structured array of 16-byte records (kind, worker, grad_id, eta) in server order."""
    cap = int(lib().synth_event_log_size(M, pushes, proto))
    out = np.zeros(cap, dtype=EVENT_DTYPE)
    n = int(lib().synth_event_log(out.ctypes.data, cap, M, pushes, order, order_param, proto,
                                  num_grads, eta, seed, stream))
    if n != cap:
        raise ValueError("synth_event_log rejected its arguments")
    return out


def make_log(records) -> np.ndarray:
    """Hand-written log from tuples ``(kind, worker[, grad_id[, eta]])``; eta < 0 means the
    server's default learning rate."""
    out = np.zeros(len(records), dtype=EVENT_DTYPE)
    for i, r in enumerate(records):
        out["kind"][i] = r[0]
        out["worker"][i] = r[1]
        out["grad_id"][i] = r[2] if len(r) > 2 else 0
        out["eta"][i] = r[3] if len(r) > 3 else -1.0
    return out


def delays(ev: np.ndarray, M: int) -> np.ndarray:
    """Delay tau of every push: how many pushes the server applied between the pushing
    worker's latest pull and this push (Section 2 of the paper: the global model moved from
    w_t to w_{t+tau} in the meantime)."""
    t = 0
    pulled_at = np.zeros(M, dtype=np.int64)
    out = []
    for kind, m in zip(ev["kind"].tolist(), ev["worker"].tolist()):
        if kind == PUSH:
            out.append(t - pulled_at[m])
            t += 1
        else:
            pulled_at[m] = t
    return np.asarray(out, dtype=np.int64)


# ----------------------------------------------------------------------------- workloads

@dataclass(frozen=True)
class Workload:
    """One replay configuration: shapes, hyper-parameters and how its inputs are drawn."""
    name: str
    n: int                      # parameter count
    M: int                      # workers
    pushes: int
    adaptive: bool
    bf16_grad: bool
    eta: float
    lam: float                  # lambda (constant variant) or lambda_0 (adaptive variant)
    mu: float = 0.0
    eps: float = 1e-7
    order: int = ORDER_UNIFORM
    order_param: float = 0.0
    proto: int = PROTO_ASYNC
    num_grads: int = 1          # size G of the cyclic gradient pool
    w0_sigma: float = 0.05
    nseg: int = 1               # gradient-scale segments (equal length, remainder in the last)
    sigma_lo_exp: float = -2.0  # per-segment std = 10^U, U ~ Unif[lo, hi]; nseg == 1: 10^lo
    sigma_hi_exp: float = -2.0
    seed: int = 0
    notes: str = field(default="", compare=False)

    @property
    def seg_len(self) -> int:
        return self.n // self.nseg if self.nseg > 1 else 0

    def sigma(self) -> np.ndarray:
        if self.nseg == 1:
            return np.asarray([10.0 ** self.sigma_lo_exp], dtype=np.float32)
        return log_uniform_sigma(self.nseg, self.sigma_lo_exp, self.sigma_hi_exp, self.seed)

    def w0(self, idx=None) -> np.ndarray:
        if idx is None:
            return normal(self.n, self.seed, STREAM_W0, self.w0_sigma)
        return normal_gather(idx, self.seed, STREAM_W0, self.w0_sigma)

    def grad(self, gid: int, idx=None) -> np.ndarray:
        """Gradient buffer `gid` of the pool: float32 values, or bfloat16 bit patterns
        (uint16) for a bf16 workload.  With `idx`: float32 values at those elements."""
        if idx is None:
            return normal(self.n, self.seed, STREAM_GRAD0 + gid, self.sigma(), self.seg_len,
                          bf16=self.bf16_grad)
        return normal_gather(idx, self.seed, STREAM_GRAD0 + gid, self.sigma(), self.seg_len,
                             through_bf16=self.bf16_grad)

    def grad_into(self, out: np.ndarray, gid: int, threads: int = 0) -> np.ndarray:
        return normal_into(out, 0, self.seed, STREAM_GRAD0 + gid, self.sigma(), self.seg_len,
                           threads)

    def log(self) -> np.ndarray:
        return event_log(self.M, self.pushes, self.order, self.proto, self.num_grads,
                         self.eta, self.seed, self.order_param)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


_WORKLOADS = {
    # constant-lambda replay at the size of the CIFAR-10 network (ResNet-20), M=4,
    # CIFAR-10 hyper-parameter lambda=0.04
    "c1_resnet20_const": Workload(
        name="c1_resnet20_const", n=272_474, M=4, pushes=2_000, adaptive=False, bf16_grad=False,
        eta=0.1, lam=0.04, order=ORDER_ROUND_ROBIN_JITTER, num_grads=2_000, w0_sigma=0.05,
        sigma_lo_exp=-2.0, sigma_hi_exp=-2.0, seed=0,
        notes="round-robin pushers with +-1 jitter; one distinct gradient per push"),
    # adaptive replay, M=8, lambda_0=2, mu=0.95 (the CIFAR-10 adaptive setting)
    "c2_adaptive_1p7m": Workload(
        name="c2_adaptive_1p7m", n=1_700_000, M=8, pushes=10_000, adaptive=True, bf16_grad=False,
        eta=0.1, lam=2.0, mu=0.95, eps=1e-7, order=ORDER_UNIFORM, num_grads=256,
        nseg=60, sigma_lo_exp=-4.0, sigma_hi_exp=-1.0, seed=0,
        notes="uniform random pusher (geometric delay, mean about M-1); cyclic pool of 256"),
    # ImageNet network size (ResNet-50), M=16 as in the paper's ImageNet run
    "c3_resnet50_adaptive": Workload(
        name="c3_resnet50_adaptive", n=25_557_032, M=16, pushes=5_000, adaptive=True,
        bf16_grad=False, eta=0.1, lam=2.0, mu=0.95, eps=1e-7, order=ORDER_UNIFORM,
        num_grads=64, nseg=161, sigma_lo_exp=-5.0, sigma_hi_exp=-1.0, seed=0,
        notes="uniform random pusher; cyclic pool of 64"),
    # large-model stress (VGG-16 size), bf16 gradients, heavy-tailed delays
    "c4_vgg16_const_bf16": Workload(
        name="c4_vgg16_const_bf16", n=138_357_544, M=32, pushes=2_000, adaptive=False,
        bf16_grad=True, eta=0.05, lam=0.04, order=ORDER_ZIPF, order_param=1.2, num_grads=32,
        sigma_lo_exp=-2.0, sigma_hi_exp=-2.0, seed=0,
        notes="Zipf(1.2) worker speeds; cyclic pool of 32 bf16 gradients"),
    "c4_vgg16_adaptive_bf16": Workload(
        name="c4_vgg16_adaptive_bf16", n=138_357_544, M=32, pushes=2_000, adaptive=True,
        bf16_grad=True, eta=0.05, lam=2.0, mu=0.95, eps=1e-7, order=ORDER_ZIPF, order_param=1.2,
        num_grads=32, sigma_lo_exp=-2.0, sigma_hi_exp=-2.0, seed=0,
        notes="Zipf(1.2) worker speeds; cyclic pool of 32 bf16 gradients"),
}


def workload(name: str) -> Workload:
    return _WORKLOADS[name]


def workload_names() -> list[str]:
    return list(_WORKLOADS)
