"""Python binding of the C-ABI server library (`include/dcasgd.h`), same names, argument
marshalling only: every step of the update runs in the library's CUDA kernels.

PyTorch is used for device memory and streams only.  There is no CPU fallback: if the shared
library cannot be loaded the import of `lib()` raises.

    srv = Server(w0, num_workers=8, adaptive=True, eta=0.1, lam=2.0, mu=0.95, eps=1e-7)
    srv.pull(3); srv.push(3, g); srv.apply_log(events, grad_pool, window_k=32)

Algorithm 2 of the paper is the server; `pull`/`push` are its two messages, `apply_log` its
repeat-loop over a recorded message log.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "csrc", "libdcasgd.so")
DEBUG_LIB_PATH = os.path.join(HERE, "csrc", "libdcasgd_checked.so")    # the -DDCASGD_DEBUG_CHECKS build

OK, EINVAL, EWORKER, EALIGN, ELOG, ECUDA, ENOMEM = range(7)
CONST, ADAPTIVE = 0, 1
F32, BF16 = 0, 1
PULL, PUSH = 0, 1
RESUME = 1
MAX_WINDOW_PUSHES, MAX_WINDOW_STORES, MAX_WINDOW_SLOTS = 640, 960, 16

# every symbol include/dcasgd.h declares
SYMBOLS = ["dcasgd_create", "dcasgd_pull", "dcasgd_push", "dcasgd_apply_log", "dcasgd_destroy",
           "dcasgd_get_step", "dcasgd_set_step", "dcasgd_get_launch_count", "dcasgd_last_error",
           "dcasgd_status_string", "dcasgd_version", "dcasgd_compile_window", "dcasgd_check_adaptive_lambda",
           "dcasgd_get_window_slot_cap", "dcasgd_debug_checks", "dcasgd_check_adaptive_lambda_grid"]


class Config(C.Structure):
    _fields_ = [("n", C.c_uint64), ("num_workers", C.c_uint32), ("variant", C.c_uint32),
                ("grad_dtype", C.c_uint32), ("eta", C.c_float), ("lambda_", C.c_float),
                ("mu", C.c_float), ("eps", C.c_float), ("flags", C.c_uint32), ("w", C.c_void_p), ("w_bak", C.c_void_p),
                ("w_bak_stride", C.c_uint64), ("ms", C.c_void_p), ("stream", C.c_void_p),
                ("v", C.c_void_p), ("beta", C.c_float), ("reserved", C.c_uint32)]


class WindowProgram(C.Structure):
    _fields_ = [("n_records", C.c_uint32), ("n_pushes", C.c_uint32), ("n_slots", C.c_uint32),
                ("n_stores", C.c_uint32), ("n_snapshot_reads", C.c_uint32), ("n_dead_pulls", C.c_uint32),
                ("grad_id", C.c_uint32 * MAX_WINDOW_PUSHES), ("eta", C.c_float * MAX_WINDOW_PUSHES),
                ("src", C.c_int32 * MAX_WINDOW_PUSHES), ("save_slot", C.c_int32 * (MAX_WINDOW_PUSHES + 1)),
                ("store_begin", C.c_uint32 * (MAX_WINDOW_PUSHES + 2)),
                ("store_worker", C.c_uint32 * MAX_WINDOW_STORES)]


class DcasgdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{status_string(status)}: {message}")
        self.status = status
        self.message = message


_lib = None


def lib() -> C.CDLL:
    """Loads csrc/libdcasgd.so (building it in-tree first if it is absent and nvcc exists)."""
    global _lib
    if _lib is None:
        # DCASGD_CHECKED_BUILD=1 selects the library whose kernels bounds-check every access
        checked = os.environ.get("DCASGD_CHECKED_BUILD", "0") == "1"
        path = DEBUG_LIB_PATH if checked else LIB_PATH
        if not os.path.exists(path):
            from . import build
            build.build_lib(debug_checks=checked)
        L = C.CDLL(path)
        u64, u32, vp = C.c_uint64, C.c_uint32, C.c_void_p
        L.dcasgd_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
        L.dcasgd_pull.argtypes = [vp, u32, vp]
        L.dcasgd_push.argtypes = [vp, u32, vp, C.c_float]
        L.dcasgd_apply_log.argtypes = [vp, vp, u64, vp, u64, u32, u32]
        L.dcasgd_destroy.argtypes = [vp]
        L.dcasgd_get_step.argtypes = [vp, C.POINTER(u64)]
        L.dcasgd_set_step.argtypes = [vp, u64]
        L.dcasgd_get_launch_count.argtypes = [vp, C.POINTER(u64)]
        L.dcasgd_compile_window.argtypes = [vp, u64, u32, u32, C.c_float, u32, C.POINTER(WindowProgram)]
        L.dcasgd_get_window_slot_cap.argtypes = [vp, C.POINTER(u32)]
        L.dcasgd_get_window_slot_cap.restype = C.c_int
        L.dcasgd_check_adaptive_lambda.argtypes = [C.c_float, C.c_float, C.c_float, vp, vp]
        L.dcasgd_check_adaptive_lambda.restype = C.c_int
        L.dcasgd_check_adaptive_lambda_grid.argtypes = [C.c_float, u32, u32, C.c_float, C.c_float, vp, vp]
        L.dcasgd_check_adaptive_lambda_grid.restype = C.c_int
        L.dcasgd_debug_checks.argtypes = [vp, vp]
        L.dcasgd_debug_checks.restype = C.c_int
        for name in ("dcasgd_create", "dcasgd_pull", "dcasgd_push", "dcasgd_apply_log", "dcasgd_destroy",
                     "dcasgd_get_step", "dcasgd_set_step", "dcasgd_get_launch_count", "dcasgd_compile_window"):
            getattr(L, name).restype = C.c_int
        L.dcasgd_last_error.restype = C.c_char_p
        L.dcasgd_status_string.restype = C.c_char_p
        L.dcasgd_status_string.argtypes = [C.c_int]
        L.dcasgd_version.restype = u32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().dcasgd_status_string(status).decode()


def last_error() -> str:
    return lib().dcasgd_last_error().decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise DcasgdError(rc, last_error())


def _ptr(x) -> int | None:
    """Address of a torch tensor / numpy array, or a raw integer address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data


# ---------------------------------------------------------------- the C calls, one to one

def dcasgd_create(n, num_workers, variant, grad_dtype, eta, lam, mu, eps, w, w_bak, w_bak_stride,
                  ms, stream=None, flags=0, v=None, beta=0.0) -> int:
    cfg = Config(n, num_workers, variant, grad_dtype, eta, lam, mu, eps, flags, _ptr(w), _ptr(w_bak),
                 w_bak_stride, _ptr(ms), stream, _ptr(v), beta, 0)
    h = C.c_void_p()
    _check(lib().dcasgd_create(C.byref(cfg), C.byref(h)))
    return h.value


def dcasgd_pull(h, m, out_w=None) -> None:
    _check(lib().dcasgd_pull(h, m, _ptr(out_w)))


def dcasgd_push(h, m, g, eta=-1.0) -> None:
    _check(lib().dcasgd_push(h, m, _ptr(g), eta))


def dcasgd_apply_log(h, ev, grad_pool, grad_stride_bytes, num_grads, window_k) -> None:
    """ev: numpy structured array of 16-byte records (host).  grad_pool: device buffer."""
    ev = np.ascontiguousarray(ev)
    assert ev.dtype.itemsize == 16
    _check(lib().dcasgd_apply_log(h, ev.ctypes.data if ev.size else None, ev.size, _ptr(grad_pool),
                                  grad_stride_bytes, num_grads, window_k))


def dcasgd_destroy(h) -> None:
    _check(lib().dcasgd_destroy(h))


def dcasgd_get_step(h) -> int:
    t = C.c_uint64()
    _check(lib().dcasgd_get_step(h, C.byref(t)))
    return t.value


def dcasgd_set_step(h, t) -> None:
    _check(lib().dcasgd_set_step(h, t))


def dcasgd_get_launch_count(h) -> int:
    t = C.c_uint64()
    _check(lib().dcasgd_get_launch_count(h, C.byref(t)))
    return t.value


def dcasgd_version() -> int:
    return int(lib().dcasgd_version())


def dcasgd_compile_window(ev, num_workers, window_k, default_eta=0.0, max_slots=0) -> WindowProgram:
    """Host only (no GPU needed): the step program of the window that starts at ev[0]."""
    ev = np.ascontiguousarray(ev)
    out = WindowProgram()
    _check(lib().dcasgd_compile_window(ev.ctypes.data if ev.size else None, ev.size, num_workers, window_k,
                                       default_eta, max_slots, C.byref(out)))
    return out


def dcasgd_get_window_slot_cap(h) -> int:
    cap = C.c_uint32()
    _check(lib().dcasgd_get_window_slot_cap(h, C.byref(cap)))
    return cap.value


def dcasgd_check_adaptive_lambda(lambda0, s_first, s_last, mismatches_dev, stream=None) -> None:
    """Adds to the device counter the number of s in [s_first, s_last] on which the two routes
    of lambda_0 / sqrt(s) differ (expected: 0)."""
    _check(lib().dcasgd_check_adaptive_lambda(lambda0, s_first, s_last, stream, _ptr(mismatches_dev)))


def dcasgd_check_adaptive_lambda_grid(a_first, a_count, a_step, s_first, s_last, mismatches_dev, stream=None) -> None:
    """The same over a grid: a_count numerators (encodings bits(a_first) + i * a_step) times every
    s in [s_first, s_last].  a in [1, 2) with step 1 and s in [1, 4) covers every significand pair."""
    _check(lib().dcasgd_check_adaptive_lambda_grid(a_first, a_count, a_step, s_first, s_last, stream, _ptr(mismatches_dev)))


def dcasgd_debug_checks(h, status_dev) -> None:
    """Checked build only: the device word that collects access violations (see dcasgd.h)."""
    _check(lib().dcasgd_debug_checks(h, _ptr(status_dev)))


def plan_log(ev, num_workers, window_k, default_eta=0.0, max_slots=0) -> list[WindowProgram]:
    """All windows of a log, as dcasgd_apply_log cuts them when max_slots is the server's
    dcasgd_get_window_slot_cap."""
    out, r = [], 0
    while r < len(ev):
        p = dcasgd_compile_window(ev[r:], num_workers, window_k, default_eta, max_slots)
        out.append(p)
        r += p.n_records
    return out


def apply_log_from_host(h, ev, host_pool, dev_pool, window_k, copy_stream, chunk: int = 8) -> int:
    """dcasgd_apply_log for a gradient pool that still sits in (pinned) host memory.

    `host_pool` and `dev_pool` are [G][row] torch tensors of the same shape and dtype.  The pool
    buffers are copied to the device on `copy_stream` in the order in which the log first uses
    them, `chunk` buffers per event, and each piece of the log is enqueued (on the current
    stream, which must be the server's) as soon as the buffers it names have arrived, so the
    transfer overlaps the replay of the earlier pieces.  Results equal one dcasgd_apply_log call
    on a resident pool.  Returns the number of host->device bytes enqueued."""
    import torch
    ev = np.ascontiguousarray(ev)
    G = host_pool.shape[0]
    stride = dev_pool.stride(0) * dev_pool.element_size()
    push_idx = np.flatnonzero(ev["kind"] == PUSH)
    gids = ev["grad_id"][push_idx]
    order, first_rec = [], []                         # buffers in first-use order, record of first use
    seen = set()
    for r, g in zip(push_idx.tolist(), gids.tolist()):
        if g not in seen:
            seen.add(g)
            order.append(g)
            first_rec.append(r)
            if len(seen) == G:
                break
    main = torch.cuda.current_stream()
    copy_stream.wait_stream(main)                     # the device pool may still be read by earlier work
    start, nbytes = 0, 0
    for c in range(0, len(order), chunk):
        with torch.cuda.stream(copy_stream):
            for g in order[c:c + chunk]:
                dev_pool[g].copy_(host_pool[g], non_blocking=True)
                nbytes += host_pool[g].numel() * host_pool.element_size()
            arrived = torch.cuda.Event()
            arrived.record(copy_stream)
        nxt = c + chunk
        end = first_rec[nxt] if nxt < len(order) else len(ev)
        main.wait_event(arrived)
        dcasgd_apply_log(h, ev[start:end], dev_pool, stride, G, window_k)
        start = end
    if start < len(ev):
        dcasgd_apply_log(h, ev[start:], dev_pool, stride, G, window_k)
    return nbytes


# ---------------------------------------------------------------- convenience wrapper

def padded_stride(n: int) -> int:
    """Backup-slab stride in floats: n rounded up to 32 floats (128-byte rows)."""
    return (n + 31) // 32 * 32


class Server:
    """Owns the torch tensors a server borrows (w, w_bak, ms) and the handle."""

    def __init__(self, w0, num_workers: int, adaptive: bool, eta: float, lam: float, mu: float = 0.0,
                 eps: float = 0.0, bf16_grad: bool = False, device="cuda", stream=None, state: dict | None = None,
                 beta: float | None = None):
        """`state` (from state_dict()) resumes a saved server instead of initialising from w0.
        `beta` (not None) selects the momentum variant with that coefficient."""
        import torch
        self.torch = torch
        self.device = torch.device(device)
        w0 = torch.as_tensor(w0 if state is None else state["w"], dtype=torch.float32).reshape(-1)
        self.n = int(w0.numel())
        self.M = int(num_workers)
        self.stride = padded_stride(self.n)
        self.w = w0.to(self.device, copy=True).contiguous()
        self.w_bak_buf = torch.empty(self.M * self.stride, dtype=torch.float32, device=self.device)
        self.ms = torch.empty(self.n, dtype=torch.float32, device=self.device) if adaptive else None
        self.v = torch.empty(self.n, dtype=torch.float32, device=self.device) if beta is not None else None
        if state is not None:
            self.w_bak_buf.view(self.M, self.stride)[:, : self.n].copy_(state["w_bak"])
            if adaptive:
                self.ms.copy_(state["ms"])
            if beta is not None:
                self.v.copy_(state["v"])
        self.bf16_grad = bool(bf16_grad)
        self.stream = stream
        if stream is not None:
            # the copies above ran on torch's current stream; the server's kernels run on `stream`
            stream.wait_stream(torch.cuda.current_stream(self.device))
        s = stream.cuda_stream if stream is not None else torch.cuda.current_stream(self.device).cuda_stream
        with torch.cuda.device(self.device):
            self.h = dcasgd_create(self.n, self.M, ADAPTIVE if adaptive else CONST, BF16 if bf16_grad else F32,
                                   eta, lam, mu, eps, self.w, self.w_bak_buf, self.stride, self.ms, s,
                                   flags=RESUME if state is not None else 0, v=self.v,
                                   beta=0.0 if beta is None else beta)
        if state is not None:
            dcasgd_set_step(self.h, int(state["t"]))

    def state_dict(self) -> dict:
        """The whole server state (w, every backup, MeanSquare, t) as host copies: a checkpoint."""
        self.torch.cuda.synchronize(self.device)
        return {"w": self.w.cpu(), "w_bak": self.w_bak.cpu(), "ms": None if self.ms is None else self.ms.cpu(),
                "v": None if self.v is None else self.v.cpu(), "t": self.step}

    @property
    def w_bak(self):
        return self.w_bak_buf.view(self.M, self.stride)[:, : self.n]

    def pull(self, m: int, out_w=None) -> None:
        dcasgd_pull(self.h, m, out_w)

    def push(self, m: int, g, eta: float = -1.0) -> None:
        dcasgd_push(self.h, m, g, eta)

    def apply_log(self, ev, grad_pool, window_k: int, grad_stride_bytes: int | None = None,
                  num_grads: int | None = None) -> None:
        """grad_pool: [G][row] device tensor (float32, or bfloat16/int16 for bf16 gradients)."""
        if grad_stride_bytes is None:
            grad_stride_bytes = grad_pool.stride(0) * grad_pool.element_size()
        if num_grads is None:
            num_grads = grad_pool.shape[0]
        dcasgd_apply_log(self.h, ev, grad_pool, grad_stride_bytes, num_grads, window_k)

    @property
    def step(self) -> int:
        return dcasgd_get_step(self.h)

    @property
    def launches(self) -> int:
        return dcasgd_get_launch_count(self.h)

    def close(self) -> None:
        if getattr(self, "h", None):
            dcasgd_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
