"""ctypes binding of the CPU checker (`dcasgd_oracle.cpp`).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package.
It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "dcasgd_oracle.cpp")
SO = os.path.join(HERE, "libdcasgd_oracle.so")

# -ffp-contract=off: no fused multiply-add; no fast-math: every operation rounds on its own.
CXXFLAGS = ["-O2", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math", "-Wall"]

PULL, PUSH = 0, 1


def build(force: bool = False, src: str = SRC, so: str = SO) -> str:
    if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
        proc = subprocess.run(["g++", *CXXFLAGS, "-o", so, src], capture_output=True, text=True)
        if proc.returncode != 0:
            raise RuntimeError("oracle build failed:\n" + proc.stderr)
    return so


def _bind(path: str) -> C.CDLL:
    L = C.CDLL(path)
    u64, u32, i32, vp = C.c_uint64, C.c_uint32, C.c_int, C.c_void_p
    for suf, real in (("f32", C.c_float), ("f64", C.c_double)):
        getattr(L, f"oracle_init_{suf}").argtypes = [u64, u32, vp, vp, vp]
        getattr(L, f"oracle_init_{suf}").restype = None
        getattr(L, f"oracle_pull_{suf}").argtypes = [u64, u32, vp, vp]
        getattr(L, f"oracle_pull_{suf}").restype = None
    L.oracle_push_f32.argtypes = [u64, u32, i32] + [C.c_float] * 4 + [vp, vp, vp, vp, i32, C.c_float, vp]
    L.oracle_push_f32.restype = None
    L.oracle_push_f64.argtypes = [u64, u32, i32] + [C.c_double] * 4 + [vp, vp, vp, vp, C.c_double, vp]
    L.oracle_push_f64.restype = None
    L.oracle_replay_f32.argtypes = [u64, u32, i32] + [C.c_float] * 4 + [vp, vp, vp, vp, u64, vp, u64, u32, i32, vp, C.c_float, vp]
    L.oracle_replay_f32.restype = i32
    L.oracle_replay_f64.argtypes = [u64, u32, i32] + [C.c_double] * 4 + [vp, vp, vp, vp, u64, vp, u64, u32, vp, C.c_double, vp]
    L.oracle_replay_f64.restype = i32
    return L


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data


class Server:
    """State of Algorithm 2 on the host: w[n], w_bak[M][n], ms[n] (adaptive), step counter t.

    dtype float32 follows the precision the GPU library computes in; float64 is used by the
    pins that compare against closed forms.
    """

    def __init__(self, w0, M: int, adaptive: bool, eta: float, lam: float, mu: float = 0.0,
                 eps: float = 0.0, dtype=np.float32, library: C.CDLL | None = None, beta: float | None = None):
        self.L = library or lib()
        self.dtype = np.dtype(dtype)
        self.suf = "f32" if self.dtype == np.float32 else "f64"
        self.n = int(np.asarray(w0).size)
        self.M = int(M)
        self.adaptive = bool(adaptive)
        self.eta, self.lam, self.mu, self.eps = eta, lam, mu, eps
        self.w = np.array(w0, dtype=self.dtype).reshape(-1).copy()
        self.w_bak = np.empty((self.M, self.n), dtype=self.dtype)
        self.ms = np.empty(self.n, dtype=self.dtype) if adaptive else None
        self.beta = 0.0 if beta is None else beta               # momentum: None = off (no velocity vector)
        self.v = None if beta is None else np.zeros(self.n, dtype=self.dtype)
        self.t = C.c_uint64(0)
        getattr(self.L, f"oracle_init_{self.suf}")(self.n, self.M, _ptr(self.w), _ptr(self.w_bak),
                                                   _ptr(self.ms))

    @property
    def step(self) -> int:
        return int(self.t.value)

    def pull(self, m: int) -> None:
        assert 0 <= m < self.M
        getattr(self.L, f"oracle_pull_{self.suf}")(self.n, m, _ptr(self.w), _ptr(self.w_bak))

    def push(self, m: int, g: np.ndarray, eta: float | None = None) -> None:
        assert 0 <= m < self.M and g.size == self.n and g.flags.c_contiguous
        e = self.eta if eta is None or eta < 0 else eta
        if self.suf == "f32":
            assert g.dtype in (np.float32, np.uint16)
            self.L.oracle_push_f32(self.n, m, int(self.adaptive), e, self.lam, self.mu, self.eps,
                                   _ptr(self.w), _ptr(self.w_bak), _ptr(self.ms), _ptr(g),
                                   int(g.dtype == np.uint16), self.beta, _ptr(self.v))
        else:
            assert g.dtype == np.float64
            self.L.oracle_push_f64(self.n, m, int(self.adaptive), e, self.lam, self.mu, self.eps,
                                   _ptr(self.w), _ptr(self.w_bak), _ptr(self.ms), _ptr(g), self.beta, _ptr(self.v))
        self.t.value += 1

    def replay(self, ev: np.ndarray, grads: np.ndarray) -> None:
        """Apply a log serially.  `grads` is a [G][n] array (float32, uint16 bfloat16 patterns,
        or float64 for a float64 server); rows may be strided (a column slice of a wider pool)."""
        assert ev.dtype.itemsize == 16 and ev.flags.c_contiguous
        assert grads.ndim == 2 and grads.shape[1] == self.n
        assert grads.strides[1] == grads.itemsize and grads.strides[0] % grads.itemsize == 0
        G = grads.shape[0]
        stride = grads.strides[0] // grads.itemsize
        if self.suf == "f32":
            assert grads.dtype in (np.float32, np.uint16)
            rc = self.L.oracle_replay_f32(self.n, self.M, int(self.adaptive), self.eta, self.lam,
                                          self.mu, self.eps, _ptr(self.w), _ptr(self.w_bak),
                                          _ptr(self.ms), _ptr(ev), ev.size, _ptr(grads), stride, G,
                                          int(grads.dtype == np.uint16), C.addressof(self.t), self.beta, _ptr(self.v))
        else:
            assert grads.dtype == np.float64
            rc = self.L.oracle_replay_f64(self.n, self.M, int(self.adaptive), self.eta, self.lam,
                                          self.mu, self.eps, _ptr(self.w), _ptr(self.w_bak),
                                          _ptr(self.ms), _ptr(ev), ev.size, _ptr(grads), stride, G,
                                          C.addressof(self.t), self.beta, _ptr(self.v))
        if rc != 0:
            raise ValueError(f"oracle rejected the log (code {rc})")
