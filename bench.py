#!/usr/bin/env python
"""Benchmark of the DC-ASGD parameter-server update on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--window-k 32]
    python bench.py --impl reference ...        # the CPU checker timed on the host cores

One STEP is one replay of the workload's whole message log through the C-ABI library:
Algorithm 2's Initialize (dcasgd_create) followed by its message loop over every logged
pull/push (dcasgd_apply_log with fused windows of `--window-k` records).  The metric is
element-updates per second = parameters x pushes / time.  Inputs are synthetic and seeded
(shapes of the paper's workloads; see paper_1609_08326_b200.synth.workload).

Printed: ONE JSON line (rank 0).  Besides the headline it carries
  roofline      the dominant kernel (fused window replay) against measured HBM copy bandwidth
  variants      the same log replayed with windows of 8 and of 256 records and unfused (one kernel per message)
  kernels       single push / single pull kernels timed on their own (50 launches each)
  workloads     the other configurations of the benchmark set (c1, c2, c4 constant and adaptive), each
                with fused windows of 32 and 8 records, one kernel per message, and the single kernels;
                a fixed small step count of their own and a clock sample each (N = 1 only)
  e2e           the same metric with host buffers: pinned host -> device copies of the model and
                the gradient pool, replay, and the model copied back, all inside the timed region
  cpu_baseline  the CPU checker on the host cores, on a bounded sample of the same workload
With N > 1 (torchrun) every rank replays the same workload on its own GPU (independent
replicas: the path has no exchange step); time is the slowest rank's, units are summed.
With --sharded the N GPUs hold ONE server instead, each a contiguous element range of it
(strong scaling: the units of the whole job are counted once).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1609_08326_b200 import accounting as acct  # noqa: E402
from paper_1609_08326_b200 import synth  # noqa: E402

METRIC = "DC-ASGD element-updates/s"
UNIT = "element-updates/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 7700.0           # B200 HBM3e datasheet figure (HGX), reported beside the measured copy peak
DEFAULT_WORKLOAD = "c3_resnet50_adaptive"

# DRAM bytes per launch measured once with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a
# smaller case of the same kernel (n = 25,557,032, pool 16, 64 pushes), stored as DRAM bytes per
# algorithmic byte of the captured launches (fp32 gradients: 4.046 GB / 4.089 GB and 3.846 GB /
# 3.885 GB; bf16 gradients: 3.016 GB / 3.067 GB and 3.625 GB / 3.680 GB) and scaled to a launch of
# the benchmark by its algorithmic bytes.  Tied to the kernel sources by hash: a changed kernel
# voids the figure (reported as null).  The kept ncu summaries of those captures give the commands.
NCU_TRAFFIC: dict[str, dict] = {
    "k_replay<adaptive,f32>": {"src": "39d5c41caf6982a4", "dram_bytes_per_algorithmic_byte": 0.9896},
    "k_replay<adaptive,bf16>": {"src": "39d5c41caf6982a4", "dram_bytes_per_algorithmic_byte": 0.9842},
}


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for f in ("kernels.cuh", "dcasgd.cu"):
        with open(os.path.join(ROOT, "paper_1609_08326_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def hbm_peak() -> tuple[float, str]:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 200 ms while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.lines: list[str] = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0])); smax.append(float(p[1])); power.append(float(p[2]))
            except ValueError:
                continue
            for name, val in zip(names, p[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # samples under load: the upper half by power draw
        if sm:
            cut = statistics.median(power)
            load = [s for s, pw in zip(sm, power) if pw >= cut] or sm
            return {"sm_mhz": statistics.median(load), "sm_max_mhz": max(smax), "power_w_max": max(power),
                    "samples": len(sm), "reasons": sorted(reasons)}
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}


# --------------------------------------------------------------------------------- inputs

def select_workload(args) -> synth.Workload:
    wl = synth.workload(args.workload)
    kw = {}
    if args.pushes:
        kw["pushes"] = args.pushes
    if args.pool:
        kw["num_grads"] = args.pool
    if args.n:
        kw["n"] = args.n
    if args.workers:
        kw["M"] = args.workers
    return wl.scaled(**kw) if kw else wl


def row_elems(n: int) -> int:
    return (n + 31) // 32 * 32


def host_inputs(wl: synth.Workload, threads: int, pin: bool):
    """w0 and the [G][row] gradient pool in (pinned) host memory, plus the event log."""
    import torch
    row = row_elems(wl.n)
    dt = torch.int16 if wl.bf16_grad else torch.float32
    pool = torch.zeros((wl.num_grads, row), dtype=dt, pin_memory=pin)
    view = pool.numpy().view(np.uint16) if wl.bf16_grad else pool.numpy()
    for k in range(wl.num_grads):
        wl.grad_into(view[k, : wl.n], k, threads)
    w0 = torch.empty(wl.n, dtype=torch.float32, pin_memory=pin)
    synth.normal_into(w0.numpy(), 0, wl.seed, synth.STREAM_W0, wl.w0_sigma, threads=threads)
    return w0, pool, view, wl.log()


def host_inputs_slice(wl: synth.Workload, lo: int, hi: int, threads: int, pin: bool):
    """The same inputs restricted to elements [lo, hi): what one rank of the sharded server needs.
    Every value is a function of (seed, stream, element index), so a rank draws its own slice."""
    import torch
    n = hi - lo
    row = row_elems(n)
    dt = torch.int16 if wl.bf16_grad else torch.float32
    pool = torch.zeros((wl.num_grads, row), dtype=dt, pin_memory=pin)
    view = pool.numpy().view(np.uint16) if wl.bf16_grad else pool.numpy()
    sigma, seg = wl.sigma(), wl.seg_len
    for k in range(wl.num_grads):
        synth.normal_into(view[k, :n], lo, wl.seed, synth.STREAM_GRAD0 + k, sigma, seg, threads)
    w0 = torch.empty(n, dtype=torch.float32, pin_memory=pin)
    synth.normal_into(w0.numpy(), lo, wl.seed, synth.STREAM_W0, wl.w0_sigma, threads=threads)
    return w0, pool, view, wl.log()


# --------------------------------------------------------------------------------- CPU arm

def steady_sample(ev, M: int, pushes: int):
    """`pushes` pushes of the log in steady state: the records after the M leading pulls, every
    push with the pull that follows it (so pushes : pulls = 1 : 1, as in the whole log)."""
    idx = np.flatnonzero(ev["kind"] == synth.PUSH)
    if len(idx) == 0:
        return ev
    pushes = max(1, min(pushes, len(idx)))
    start, last = int(idx[0]), int(idx[pushes - 1])
    end = last + 2 if last + 1 < len(ev) and ev["kind"][last + 1] == synth.PULL else last + 1
    return ev[start:end]


def sample_log(ev, pushes: int):
    """Prefix of the log that holds `pushes` pushes."""
    idx = np.flatnonzero(ev["kind"] == synth.PUSH)
    if pushes >= len(idx):
        return ev
    return ev[: idx[pushes - 1] + 2] if idx[pushes - 1] + 2 <= len(ev) else ev[: idx[pushes - 1] + 1]


def oracle_seconds(wl: synth.Workload, ev, w0_np, pool_np, threads: int) -> float:
    """Seconds the CPU checker takes to replay `ev` over the whole vector: its unchanged replay
    function called on disjoint element ranges from `threads` host threads.  Every thread builds
    its own server state (so the pages it works on are first touched by it), all threads then
    meet at a barrier, and the clock runs from that barrier to the last thread's return."""
    import oracle
    f = np.float32
    bounds = np.linspace(0, wl.n, threads + 1).astype(np.int64)
    gate = threading.Barrier(threads + 1)
    errors: list[BaseException] = []

    def work(lo: int, hi: int) -> None:
        try:
            srv = oracle.Server(w0_np[lo:hi], wl.M, wl.adaptive, f(wl.eta), f(wl.lam), f(wl.mu), f(wl.eps))
            cols = pool_np[:, lo:hi]
        except BaseException as e:                       # let the barrier pass, report afterwards
            errors.append(e)
            gate.wait()
            return
        gate.wait()
        srv.replay(ev, cols)

    ths = [threading.Thread(target=work, args=(int(lo), int(hi))) for lo, hi in zip(bounds[:-1], bounds[1:])]
    for t in ths:
        t.start()
    gate.wait()
    t0 = time.perf_counter()
    for t in ths:
        t.join()
    dt = time.perf_counter() - t0
    if errors:
        raise errors[0]
    return dt


def oracle_rate(wl: synth.Workload, ev, w0_np, pool_np, threads: int, target_s: float, max_pushes: int | None = None):
    """Times the checker on a steady-state sample sized for about `target_s` seconds (at least one
    second, so that thread start-up does not show).  Returns (element-updates/s, pushes, seconds)."""
    probe = steady_sample(ev, wl.M, 4 if threads > 1 else 1)
    p_probe = int(np.sum(probe["kind"] == synth.PUSH))
    oracle_seconds(wl, probe, w0_np, pool_np, threads)               # warms caches and the thread pool of the OS
    dt = oracle_seconds(wl, probe, w0_np, pool_np, threads)
    per_push = max(dt / p_probe, 1e-9)
    pushes = int(max(1, min(max_pushes or wl.pushes, wl.pushes, round(target_s / per_push))))
    sample = steady_sample(ev, wl.M, pushes)
    p = int(np.sum(sample["kind"] == synth.PUSH))
    dt = oracle_seconds(wl, sample, w0_np, pool_np, threads)
    return wl.n * p / dt, p, dt


def cpu_baseline(wl, ev, w0_np, pool_np, target_s: float = 12.0) -> dict:
    cores = os.cpu_count() or 1
    value, p, dt = oracle_rate(wl, ev, w0_np, pool_np, cores, target_s)
    value1, p1, dt1 = oracle_rate(wl, ev, w0_np, pool_np, 1, target_s * 0.75)
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{p} consecutive pushes (each with the pull that follows it, after the {wl.M} leading pulls) of the "
                      f"{wl.name} log on the full vector n={wl.n}, {cores} host threads over disjoint element ranges, {dt:.1f} s",
            "single_thread_value": value1, "single_thread_sample": f"{p1} pushes, {dt1:.1f} s"}


def run_reference(args) -> None:
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = select_workload(args)
    cores = os.cpu_count() or 1
    log = wl.log()
    # a step is a steady-state sample of about a second (or --ref-pushes pushes); a bounded part
    # of the gradient pool is enough for it
    budget = args.ref_pushes or min(wl.pushes, 4 * wl.num_grads)
    ev = steady_sample(log, wl.M, budget)
    G = int(ev["grad_id"].max()) + 1
    small = wl.scaled(num_grads=max(G, 1))
    w0, pool, view, _ = host_inputs(small, cores, pin=False)
    if not args.ref_pushes:
        _, p_cal, dt_cal = oracle_rate(small, ev, w0.numpy(), view, cores, 1.0, max_pushes=budget)
        ev = steady_sample(log, wl.M, max(1, min(budget, int(round(p_cal * max(1.0, 1.0 / dt_cal))))))
    p = int(np.sum(ev["kind"] == synth.PUSH))
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_seconds(small, ev, w0.numpy(), view, cores)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = wl.n * p * len(times) / total
    sample = (f"each step = {p} consecutive pushes (each with the pull that follows it, after the {wl.M} leading pulls) "
              f"of the {wl.name} log on the full vector n={wl.n}, {cores} host threads over disjoint element ranges")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, args, sample_note=sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def fits_l2(wl) -> bool:
    return wl.n * 4 * 3 <= 126e6


def config_of(wl, args, sample_note: str | None = None) -> dict:
    c = {"workload": wl.name, "n": wl.n, "workers": wl.M, "pushes": wl.pushes, "grad_pool": wl.num_grads,
         "variant": "adaptive" if wl.adaptive else "constant", "grad_dtype": "bf16" if wl.bf16_grad else "f32",
         "eta": wl.eta, "lambda": wl.lam, "mu": wl.mu, "eps": wl.eps, "window_k": args.window_k,
         "parallelism": f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU",
         "l2": "working set fits L2; L2 flushed between steps" if fits_l2(wl) else "inputs larger than L2 (no flush)"}
    if sample_note:
        c["sample"] = sample_note
    return c


# --------------------------------------------------------------------------------- GPU arm

class GpuWorkload:
    """One workload resident on the device, and the timed legs over it.  Every leg goes through
    the C-ABI binding; time is taken with CUDA events on the stream the library launches on."""

    def __init__(self, wl, local: int, world: int, dist, gen_threads: int, host=None, need_out: bool = True):
        import torch
        from paper_1609_08326_b200 import binding as B
        self.torch, self.B, self.wl, self.world, self.dist = torch, B, wl, world, dist
        self.w0_h, self.pool_h, self.pool_view, self.ev = host if host is not None else host_inputs(wl, gen_threads, pin=True)
        self.n_push = int(np.sum(self.ev["kind"] == synth.PUSH))
        self.n_pull = len(self.ev) - self.n_push
        self.units = float(wl.n) * self.n_push
        dev = torch.device("cuda", local)
        gdt = torch.int16 if wl.bf16_grad else torch.float32
        self.stride = B.padded_stride(wl.n)
        self.w = torch.empty(wl.n, dtype=torch.float32, device=dev)
        self.w0_d = torch.empty(wl.n, dtype=torch.float32, device=dev)
        self.w_bak = torch.empty(wl.M * self.stride, dtype=torch.float32, device=dev)
        self.ms = torch.empty(wl.n, dtype=torch.float32, device=dev) if wl.adaptive else None
        self.pool = torch.empty(self.pool_h.shape, dtype=gdt, device=dev)
        self.w_out = torch.empty(wl.n, dtype=torch.float32, pin_memory=True) if need_out else None
        self.gstride = self.pool.stride(0) * self.pool.element_size()
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if fits_l2(wl) else None
        self.w0_d.copy_(self.w0_h)
        self.pool.copy_(self.pool_h)
        torch.cuda.synchronize()
        self.stream = torch.cuda.current_stream().cuda_stream
        self.copy_stream = torch.cuda.Stream()
        self.launches = 0
        self.peak, self.peak_kind = hbm_peak()
        h = self.create()
        self.slot_cap = B.dcasgd_get_window_slot_cap(h)      # cut the log exactly as dcasgd_apply_log does
        B.dcasgd_destroy(h)
        self._plans: dict[int, tuple[int, int]] = {}

    def host(self):
        return self.w0_h, self.pool_h, self.pool_view, self.ev

    def create(self):
        B, wl = self.B, self.wl
        return B.dcasgd_create(wl.n, wl.M, B.ADAPTIVE if wl.adaptive else B.CONST, B.BF16 if wl.bf16_grad else B.F32,
                               wl.eta, wl.lam, wl.mu, wl.eps, self.w, self.w_bak, self.stride, self.ms, self.stream)

    def replay_steps(self, window_k: int, steps: int, warmup: int, host_io: bool = False):
        """Times `steps` whole-log replays; returns (total ms, replay-only ms, launches per step).
        Each step starts from the configured w0: it is restored from a device copy before the
        step's first event (with host_io the step itself copies it from pinned host memory)."""
        torch, B, wl = self.torch, self.B, self.wl
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
                torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        per_step = 0
        for i in range(warmup + steps):
            if self.flush is not None:
                self.flush.fill_(i & 0xFF)
            if not host_io:
                self.w.copy_(self.w0_d)
            if i == warmup:
                if self.world > 1:
                    self.dist.barrier()
                torch.cuda.synchronize()
            if i >= warmup:
                evs[i - warmup][0].record()
            if host_io:
                self.w.copy_(self.w0_h, non_blocking=True)
            h = self.create()
            if i >= warmup:
                evs[i - warmup][1].record()
            if host_io:
                B.apply_log_from_host(h, self.ev, self.pool_h, self.pool, window_k, self.copy_stream)
            else:
                B.dcasgd_apply_log(h, self.ev, self.pool, self.gstride, wl.num_grads, window_k)
            per_step = B.dcasgd_get_launch_count(h)
            B.dcasgd_destroy(h)
            if host_io:
                self.w_out.copy_(self.w, non_blocking=True)
            if i >= warmup:
                evs[i - warmup][2].record()
                self.launches += per_step
        torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
        total = sum(a.elapsed_time(c) for a, _, c in evs)
        replay = sum(b.elapsed_time(c) for _, b, c in evs)
        return total, replay, per_step

    def plan(self, window_k: int) -> tuple[int, int]:
        """(kernel launches, algorithmic bytes) of one replay of the log at this window size."""
        if window_k not in self._plans:
            wl = self.wl
            if window_k == 1:
                self._plans[1] = (len(self.ev), acct.unfused_log_bytes(self.n_push, self.n_pull, wl.adaptive, wl.bf16_grad) * wl.n)
            else:
                progs = self.B.plan_log(self.ev, wl.M, window_k, wl.eta, self.slot_cap)
                per = [acct.window_bytes(p, wl.adaptive, wl.bf16_grad) for p in progs]
                self._plans[window_k] = (sum(1 for b in per if b), sum(per) * wl.n)
        return self._plans[window_k]

    def leg(self, window_k: int, steps: int, warmup: int) -> dict:
        """One timed leg as a dictionary (device-resident inputs)."""
        t_ms, r_ms, per_step = self.replay_steps(window_k, steps, warmup)
        launches, nbytes = self.plan(window_k)
        gbs = nbytes * steps / (r_ms * 1e-3) / 1e9
        return {"value": self.units * steps / (t_ms * 1e-3), "unit": UNIT, "ms_per_step": t_ms / steps,
                "launches_per_step": per_step, "avg_launch_ms": r_ms / (steps * max(1, launches)),
                "achieved_gbs": gbs, "frac": gbs / self.peak, "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                "bytes_per_element_per_push": nbytes / self.units}

    def single_kernels(self, reps: int = 50) -> dict:
        """dcasgd_push / dcasgd_pull on their own: `reps` launches each, rotating workers and pool buffers."""
        torch, B, wl = self.torch, self.B, self.wl
        self.w.copy_(self.w0_d)
        h = self.create()
        kern = {}
        for name, fn, bpe in (
                ("k_push", lambda i: B.dcasgd_push(h, i % wl.M, self.pool[i % wl.num_grads], -1.0), acct.push_bytes(wl.adaptive, wl.bf16_grad)),
                ("k_pull", lambda i: B.dcasgd_pull(h, i % wl.M, None), acct.pull_bytes())):
            for i in range(5):
                fn(i)
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if self.flush is not None:
                self.flush.fill_(1)
            torch.cuda.synchronize()
            a.record()
            for i in range(reps):
                fn(5 + i)
            b_.record()
            torch.cuda.synchronize()
            ms_ = a.elapsed_time(b_) / reps
            gbs = bpe * wl.n / (ms_ * 1e-3) / 1e9
            kern[name] = {"avg_launch_ms": ms_, "bytes_per_element": bpe, "achieved_gbs": gbs, "frac": gbs / self.peak,
                          "frac_of_nominal": gbs / NOMINAL_HBM_GBS, "elements_per_s": wl.n / (ms_ * 1e-3)}
            self.launches += reps
        B.dcasgd_destroy(h)
        return kern

    def close(self) -> None:
        self.torch.cuda.synchronize()
        for name in ("w", "w0_d", "w_bak", "ms", "pool", "w_out", "flush", "w0_h", "pool_h", "pool_view"):
            setattr(self, name, None)
        self.torch.cuda.empty_cache()


# the other configurations of the benchmark set, each with a step count of its own (independent of
# --steps) sized so that the whole section takes about a minute: (timed steps, window sizes)
OTHER_WORKLOADS = {
    "c1_resnet20_const": (20, (32, 8, 256, 1280, 1)),
    "c2_adaptive_1p7m": (6, (32, 8, 256, 1280, 1)),
    "c4_vgg16_const_bf16": (2, (32, 8, 1)),
    "c4_vgg16_adaptive_bf16": (2, (32, 8, 1)),
}
OTHER_WARMUP = 3


def other_workloads(local: int, gen_threads: int) -> dict:
    """Every other configuration: fused windows, one kernel per message, and the single kernels."""
    out, host, host_key = {}, None, None
    for name, (steps, ks) in OTHER_WORKLOADS.items():
        wl = synth.workload(name)
        key = (wl.n, wl.seed, wl.bf16_grad, wl.num_grads, wl.nseg, wl.sigma_lo_exp, wl.sigma_hi_exp, wl.M, wl.pushes,
               wl.order, wl.order_param, wl.w0_sigma)
        sampler = ClockSampler(local)
        g = GpuWorkload(wl, local, 1, None, gen_threads, host=host if key == host_key else None, need_out=False)
        entry = {"n": wl.n, "workers": wl.M, "pushes": wl.pushes, "grad_pool": wl.num_grads,
                 "variant": "adaptive" if wl.adaptive else "constant", "grad_dtype": "bf16" if wl.bf16_grad else "f32",
                 "steps": steps, "warmup": OTHER_WARMUP,
                 "l2": "working set fits L2; L2 flushed between steps" if fits_l2(wl) else "inputs larger than L2 (no flush)"}
        for k in ks:
            entry["unfused_k1" if k == 1 else f"fused_k{k}"] = g.leg(k, steps, OTHER_WARMUP)
        entry.update(g.single_kernels())
        entry["clocks"] = sampler.stop()
        host, host_key = g.host(), key
        g.close()
        out[name] = entry
    return out


def run_sharded(args, wl, rank: int, local: int, world: int, dist, gen_threads: int) -> None:
    """Strong scaling: ONE server whose parameter vector is cut into contiguous element ranges, one
    per GPU (paper_1609_08326_b200.sharded).  Every rank replays the whole log on its own range
    with the unchanged library; the update needs no exchange.  The model a pulling worker receives
    is the all-gather of the shards, timed separately."""
    import torch
    from paper_1609_08326_b200 import sharded
    lo, hi = sharded.shard_range(wl.n, world, rank)
    local_wl = wl.scaled(n=hi - lo)
    g = GpuWorkload(local_wl, local, world, dist, gen_threads, host=host_inputs_slice(wl, lo, hi, gen_threads, pin=True), need_out=False)
    sampler = ClockSampler(local) if rank == 0 else None
    K, W = args.steps, args.warmup
    total_ms, replay_ms, per_step = g.replay_steps(args.window_k, K, W)
    max_ms, tot_units = acct.aggregate_over_ranks(total_ms, g.units * K, dist)
    launches, nbytes = g.plan(args.window_k)
    gbs = nbytes * K / (replay_ms * 1e-3) / 1e9
    # the worker's view of the model: all-gather of the shards into this rank's memory
    buf = torch.empty(world * sharded.chunk_elems(wl.n, world), dtype=torch.float32, device=g.w.device)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 10
    for i in range(3 + reps):
        if i == 3:
            torch.cuda.synchronize()
            a.record()
        sharded.gather_model(g.w, wl.n, world, dist, out=buf)
    b.record()
    torch.cuda.synchronize()
    gather_ms, _ = acct.aggregate_over_ranks(a.elapsed_time(b) / reps, 0.0, dist)
    cfg = config_of(wl, args)
    cfg["parallelism"] = f"element-range shards x{world} (contiguous, 32-element aligned; no collective in the update)"
    cfg["shard_elements"] = hi - lo
    out = {"metric": METRIC, "value": tot_units / (max_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": max_ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
           "data": "synthetic", "config": cfg,
           "roofline": {"bound": "hbm", "kernel": "k_replay (this rank's shard)", "achieved": gbs, "peak": g.peak, "unit": "GB/s",
                        "frac": gbs / g.peak, "peak_kind": f"of {g.peak_kind}", "frac_of_nominal": gbs / NOMINAL_HBM_GBS, "traffic": None,
                        "launches_per_step": launches, "avg_launch_ms": replay_ms / (K * max(1, launches))},
           "pull_allgather": {"ms": gather_ms, "model_bytes": wl.n * 4,
                              "received_gbs_per_gpu": wl.n * 4 * (world - 1) / max(1, world) / (gather_ms * 1e-3) / 1e9},
           "gpu_launches": g.launches}
    if sampler is not None:
        out["clocks"] = sampler.stop()
    g.close()
    if rank == 0:
        print(json.dumps(out))


def run_b200(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_1609_08326_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()                                          # fail loudly if the CUDA library is missing

    wl = select_workload(args)
    cores = os.cpu_count() or 1
    gen_threads = max(1, cores // world)
    if args.sharded:
        run_sharded(args, wl, rank, local, world, dist if world > 1 else None, gen_threads)
        if world > 1:
            dist.destroy_process_group()
        return
    g = GpuWorkload(wl, local, world, dist if world > 1 else None, gen_threads)
    sampler = ClockSampler(local) if rank == 0 else None
    K, W = args.steps, args.warmup

    # headline: fused windows of --window-k records, inputs resident in HBM
    total_ms, replay_ms, per_step = g.replay_steps(args.window_k, K, W)
    headline_launches = g.launches
    max_ms, tot_units = acct.aggregate_over_ranks(total_ms, g.units * K, dist if world > 1 else None)
    value = tot_units / (max_ms * 1e-3)

    win_launches, win_bytes = g.plan(args.window_k)
    peak, peak_kind = g.peak, g.peak_kind
    avg_launch_ms = replay_ms / (K * max(1, win_launches))
    achieved = (win_bytes / max(1, win_launches)) / (avg_launch_ms * 1e-3) / 1e9
    kname = f"k_replay<{'adaptive' if wl.adaptive else 'const'},{'bf16' if wl.bf16_grad else 'f32'}>"
    traffic = None
    tr = NCU_TRAFFIC.get(kname)
    if tr and tr.get("src") == kernel_source_hash():
        traffic = tr["dram_bytes_per_algorithmic_byte"] * (win_bytes / max(1, win_launches))
    roofline = {"bound": "hbm", "kernel": kname, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                "nominal_peak": NOMINAL_HBM_GBS, "traffic": traffic,
                "launches_per_step": win_launches, "avg_launch_ms": avg_launch_ms,
                "algorithmic_bytes_per_launch": win_bytes / max(1, win_launches),
                "bytes_per_element_per_push": win_bytes / g.units}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": max_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32", "data": "synthetic", "config": config_of(wl, args), "roofline": roofline}

    if not args.headline_only:
        variants = {}
        for name, wk in (("fused_k8", 8), ("fused_k256", 256), ("unfused_k1", 1)):
            if wk != args.window_k:
                variants[name] = g.leg(wk, K, W)
        out["variants"] = variants
        out["kernels"] = g.single_kernels()

        # end to end: host buffers, copies inside the timed region
        e_ms, _, _ = g.replay_steps(args.window_k, K, W, host_io=True)
        e_max, e_units = acct.aggregate_over_ranks(e_ms, g.units * K, dist if world > 1 else None)
        out["e2e"] = {"value": e_units / (e_max * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": int(g.w0_h.numel() * 4 + g.pool_h.numel() * g.pool_h.element_size()),
                      "d2h_bytes_per_step": int(g.w_out.numel() * 4), "ms_per_step": e_max / K,
                      "what": "pinned host w0 -> device, dcasgd_create, gradient pool pinned host -> device on a copy stream "
                              "overlapped with dcasgd_apply_log piece by piece (binding.apply_log_from_host), w -> pinned host"}

    out["gpu_launches"] = headline_launches
    if sampler is not None:
        out["clocks"] = sampler.stop()

    full = rank == 0 and world == 1 and not args.headline_only
    if full and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, g.ev, g.w0_h.numpy(), g.pool_view)
    g.close()
    if full and not args.no_workloads and args.workload == DEFAULT_WORKLOAD and not (args.pushes or args.pool or args.n or args.workers):
        out["workloads"] = other_workloads(local, gen_threads)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=synth.workload_names())
    ap.add_argument("--window-k", type=int, default=32)
    ap.add_argument("--pushes", type=int, default=0, help="shorten the log (profiling runs)")
    ap.add_argument("--pool", type=int, default=0, help="shrink the gradient pool (profiling runs)")
    ap.add_argument("--n", type=int, default=0, help="override the parameter count (profiling runs)")
    ap.add_argument("--workers", type=int, default=0, help="override the worker count (profiling runs)")
    ap.add_argument("--ref-pushes", type=int, default=0,
                    help="pushes per step of the reference arm (0: as many as take about one second)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the section that times the other configurations")
    ap.add_argument("--headline-only", action="store_true", help="skip variants, single kernels, e2e, CPU baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sharded", action="store_true",
                    help="N GPUs hold ONE server, cut into element ranges (strong scaling) instead of N replicas")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
