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
  e2e           the same metric with host buffers: pinned host -> device copies of the model and
                the gradient pool, replay, and the model copied back, all inside the timed region
  cpu_baseline  the CPU checker on the host cores, on a bounded sample of the same workload
With N > 1 (torchrun) every rank replays the same workload on its own GPU (independent
replicas: the path has no exchange step); time is the slowest rank's, units are summed.
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

# DRAM bytes per launch measured once with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a
# smaller case of the same kernel (n as c3, pool 16, 64 pushes), stored as DRAM bytes per algorithmic
# byte of the captured launches (4.044 GB / 4.089 GB and 3.842 GB / 3.885 GB) and scaled to a launch
# of the benchmark by its algorithmic bytes.  Tied to the kernel sources by hash: a changed kernel
# voids the figure (reported as null).  Summary: profiles/k_replay_adaptive_f32_c3_window32.md
NCU_TRAFFIC: dict[str, dict] = {
    "k_replay<adaptive,f32>": {"src": "e0f806aecbe4ea5e", "dram_bytes_per_algorithmic_byte": 0.9895},
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


# --------------------------------------------------------------------------------- CPU arm

def oracle_all_cores(wl: synth.Workload, ev, w0_np, pool_np, threads: int) -> float:
    """Seconds the CPU checker takes to replay `ev` over the whole vector, its unchanged replay
    function called on disjoint element ranges from `threads` host threads."""
    import oracle
    f = np.float32
    bounds = np.linspace(0, wl.n, threads + 1).astype(np.int64)
    servers = [oracle.Server(w0_np[lo:hi], wl.M, wl.adaptive, f(wl.eta), f(wl.lam), f(wl.mu), f(wl.eps))
               for lo, hi in zip(bounds[:-1], bounds[1:])]
    cols = [pool_np[:, lo:hi] for lo, hi in zip(bounds[:-1], bounds[1:])]
    ths = [threading.Thread(target=s.replay, args=(ev, c)) for s, c in zip(servers, cols)]
    t0 = time.perf_counter()
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    return time.perf_counter() - t0


def sample_log(ev, pushes: int):
    """Prefix of the log that holds `pushes` pushes."""
    idx = np.flatnonzero(ev["kind"] == synth.PUSH)
    if pushes >= len(idx):
        return ev
    return ev[: idx[pushes - 1] + 2] if idx[pushes - 1] + 2 <= len(ev) else ev[: idx[pushes - 1] + 1]


def cpu_baseline(wl, ev, w0_np, pool_np, target_s: float = 30.0) -> dict:
    cores = os.cpu_count() or 1
    probe = sample_log(ev, 8)
    p_probe = int(np.sum(probe["kind"] == synth.PUSH))
    oracle_all_cores(wl, probe, w0_np, pool_np, cores)              # first touch of the pages
    dt = oracle_all_cores(wl, probe, w0_np, pool_np, cores)
    rate = wl.n * p_probe / dt
    pushes = int(max(4, min(wl.pushes, target_s * rate / wl.n)))
    sample = sample_log(ev, pushes)
    p = int(np.sum(sample["kind"] == synth.PUSH))
    dt = oracle_all_cores(wl, sample, w0_np, pool_np, cores)
    one = sample_log(ev, max(1, pushes // max(1, cores // 2)))
    p1 = int(np.sum(one["kind"] == synth.PUSH))
    dt1 = oracle_all_cores(wl, one, w0_np, pool_np, 1)
    return {"value": wl.n * p / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {p} pushes (with their pulls) of the {wl.name} log on the full vector n={wl.n}, "
                      f"{cores} host threads over disjoint element ranges, {dt:.1f} s",
            "single_thread_value": wl.n * p1 / dt1, "single_thread_sample": f"first {p1} pushes, {dt1:.1f} s"}


def run_reference(args) -> None:
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = select_workload(args)
    cores = os.cpu_count() or 1
    # a bounded gradient pool is enough for a bounded sample of the log
    sample_pushes = args.ref_pushes
    ev = sample_log(wl.log(), sample_pushes)
    p = int(np.sum(ev["kind"] == synth.PUSH))
    G = int(ev["grad_id"].max()) + 1
    small = wl.scaled(num_grads=max(G, 1))
    w0, pool, view, _ = host_inputs(small, cores, pin=False)
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_all_cores(small, ev, w0.numpy(), view, cores)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = wl.n * p * len(times) / total
    sample = (f"each step = first {p} pushes (with their pulls) of the {wl.name} log on the full vector n={wl.n}, "
              f"{cores} host threads over disjoint element ranges")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, args, sample_note=sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def config_of(wl, args, sample_note: str | None = None) -> dict:
    c = {"workload": wl.name, "n": wl.n, "workers": wl.M, "pushes": wl.pushes, "grad_pool": wl.num_grads,
         "variant": "adaptive" if wl.adaptive else "constant", "grad_dtype": "bf16" if wl.bf16_grad else "f32",
         "eta": wl.eta, "lambda": wl.lam, "mu": wl.mu, "eps": wl.eps, "window_k": args.window_k,
         "parallelism": f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU",
         "l2": "inputs larger than L2 (no flush)" if wl.n * 4 * 3 > 126e6 else "working set fits L2; L2 flushed between steps"}
    if sample_note:
        c["sample"] = sample_note
    return c


# --------------------------------------------------------------------------------- GPU arm

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
    w0_h, pool_h, pool_view, ev = host_inputs(wl, gen_threads, pin=True)
    n_push = int(np.sum(ev["kind"] == synth.PUSH))
    n_pull = len(ev) - n_push
    units = float(wl.n) * n_push
    gdt = torch.int16 if wl.bf16_grad else torch.float32

    dev = torch.device("cuda", local)
    stride = B.padded_stride(wl.n)
    w = torch.empty(wl.n, dtype=torch.float32, device=dev)
    w_bak = torch.empty(wl.M * stride, dtype=torch.float32, device=dev)
    ms = torch.empty(wl.n, dtype=torch.float32, device=dev) if wl.adaptive else None
    pool = torch.empty(pool_h.shape, dtype=gdt, device=dev)
    w_out = torch.empty(wl.n, dtype=torch.float32, pin_memory=True)
    gstride = pool.stride(0) * pool.element_size()
    flush = None
    small = wl.n * 4 * 3 <= 126e6
    if small:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    w.copy_(w0_h)
    pool.copy_(pool_h)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    copy_stream = torch.cuda.Stream()

    def create():
        return B.dcasgd_create(wl.n, wl.M, B.ADAPTIVE if wl.adaptive else B.CONST, B.BF16 if wl.bf16_grad else B.F32,
                               wl.eta, wl.lam, wl.mu, wl.eps, w, w_bak, stride, ms, stream)

    launches = 0

    def replay_steps(window_k: int, steps: int, warmup: int, host_io: bool = False):
        """Times `steps` whole-log replays; returns (total ms, replay-only ms, launches per step)."""
        nonlocal launches
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
                torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        per_step = 0
        for i in range(warmup + steps):
            if flush is not None:
                flush.fill_(i & 0xFF)
            if i == warmup:
                if world > 1:
                    dist.barrier()
                torch.cuda.synchronize()
            if i >= warmup:
                evs[i - warmup][0].record()
            if host_io:
                w.copy_(w0_h, non_blocking=True)
            h = create()
            if i >= warmup:
                evs[i - warmup][1].record()
            if host_io:
                B.apply_log_from_host(h, ev, pool_h, pool, window_k, copy_stream)
            else:
                B.dcasgd_apply_log(h, ev, pool, gstride, wl.num_grads, window_k)
            per_step = B.dcasgd_get_launch_count(h)
            B.dcasgd_destroy(h)
            if host_io:
                w_out.copy_(w, non_blocking=True)
            if i >= warmup:
                evs[i - warmup][2].record()
                launches += per_step
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        total = sum(a.elapsed_time(c) for a, _, c in evs)
        replay = sum(b.elapsed_time(c) for _, b, c in evs)
        return total, replay, per_step

    sampler = ClockSampler(local) if rank == 0 else None
    K, W = args.steps, args.warmup

    # headline: fused windows of --window-k records, inputs resident in HBM
    total_ms, replay_ms, per_step = replay_steps(args.window_k, K, W)
    headline_launches = launches
    max_ms, tot_units = acct.aggregate_over_ranks(total_ms, units * K, dist if world > 1 else None)
    value = tot_units / (max_ms * 1e-3)

    h = create()
    slot_cap = B.dcasgd_get_window_slot_cap(h)       # cut the log exactly as dcasgd_apply_log does
    B.dcasgd_destroy(h)
    progs = B.plan_log(ev, wl.M, args.window_k, wl.eta, slot_cap)
    win_launches = sum(1 for p in progs if acct.window_bytes(p, wl.adaptive, wl.bf16_grad))
    win_bytes = sum(acct.window_bytes(p, wl.adaptive, wl.bf16_grad) for p in progs) * wl.n
    peak, peak_kind = hbm_peak()
    avg_launch_ms = replay_ms / (K * max(1, win_launches))
    achieved = (win_bytes / max(1, win_launches)) / (avg_launch_ms * 1e-3) / 1e9
    kname = f"k_replay<{'adaptive' if wl.adaptive else 'const'},{'bf16' if wl.bf16_grad else 'f32'}>"
    traffic = None
    tr = NCU_TRAFFIC.get(kname)
    if tr and tr.get("src") == kernel_source_hash():
        traffic = tr["dram_bytes_per_algorithmic_byte"] * (win_bytes / max(1, win_launches))
    roofline = {"bound": "hbm", "kernel": kname, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "launches_per_step": win_launches, "avg_launch_ms": avg_launch_ms,
                "algorithmic_bytes_per_launch": win_bytes / max(1, win_launches),
                "bytes_per_element_per_push": win_bytes / units}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": max_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32", "data": "synthetic", "config": config_of(wl, args), "roofline": roofline}

    if not args.headline_only:
        variants = {}
        for name, wk in (("fused_k8", 8), ("fused_k256", 256), ("unfused_k1", 1)):
            if wk == args.window_k:
                continue
            t_ms, r_ms, ps = replay_steps(wk, K, W)
            if wk == 1:
                b = acct.unfused_log_bytes(n_push, n_pull, wl.adaptive, wl.bf16_grad) * wl.n
            else:
                b = sum(acct.window_bytes(p, wl.adaptive, wl.bf16_grad) for p in B.plan_log(ev, wl.M, wk, wl.eta, slot_cap)) * wl.n
            variants[name] = {"value": units * K / (t_ms * 1e-3), "unit": UNIT, "ms_per_step": t_ms / K,
                              "launches_per_step": ps, "achieved_gbs": b * K / (r_ms * 1e-3) / 1e9,
                              "frac": b * K / (r_ms * 1e-3) / 1e9 / peak, "bytes_per_element_per_push": b / units}
        out["variants"] = variants

        # single kernels on their own: 50 launches each, rotating workers and pool buffers
        h = create()
        kern = {}
        for name, fn, bpe in (
                ("k_push", lambda i: B.dcasgd_push(h, i % wl.M, pool[i % wl.num_grads], -1.0), acct.push_bytes(wl.adaptive, wl.bf16_grad)),
                ("k_pull", lambda i: B.dcasgd_pull(h, i % wl.M, None), acct.pull_bytes())):
            reps = 50
            for i in range(5):
                fn(i)
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if flush is not None:
                flush.fill_(1)
            torch.cuda.synchronize()
            a.record()
            for i in range(reps):
                fn(5 + i)
            b_.record()
            torch.cuda.synchronize()
            ms_ = a.elapsed_time(b_) / reps
            gbs = bpe * wl.n / (ms_ * 1e-3) / 1e9
            kern[name] = {"avg_launch_ms": ms_, "bytes_per_element": bpe, "achieved_gbs": gbs, "frac": gbs / peak,
                          "elements_per_s": wl.n / (ms_ * 1e-3)}
            launches += reps
        B.dcasgd_destroy(h)
        out["kernels"] = kern

        # end to end: host buffers, copies inside the timed region
        e_ms, _, _ = replay_steps(args.window_k, K, W, host_io=True)
        e_max, e_units = acct.aggregate_over_ranks(e_ms, units * K, dist if world > 1 else None)
        out["e2e"] = {"value": e_units / (e_max * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": int(w0_h.numel() * 4 + pool_h.numel() * pool_h.element_size()),
                      "d2h_bytes_per_step": int(w_out.numel() * 4), "ms_per_step": e_max / K,
                      "what": "pinned host w0 -> device, dcasgd_create, gradient pool pinned host -> device on a copy stream "
                              "overlapped with dcasgd_apply_log piece by piece (binding.apply_log_from_host), w -> pinned host"}

    out["gpu_launches"] = headline_launches
    if sampler is not None:
        out["clocks"] = sampler.stop()

    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.headline_only:
        out["cpu_baseline"] = cpu_baseline(wl, ev, w0_h.numpy(), pool_view)
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
    ap.add_argument("--workload", default="c3_resnet50_adaptive", choices=synth.workload_names())
    ap.add_argument("--window-k", type=int, default=32)
    ap.add_argument("--pushes", type=int, default=0, help="shorten the log (profiling runs)")
    ap.add_argument("--pool", type=int, default=0, help="shrink the gradient pool (profiling runs)")
    ap.add_argument("--n", type=int, default=0, help="override the parameter count (profiling runs)")
    ap.add_argument("--workers", type=int, default=0, help="override the worker count (profiling runs)")
    ap.add_argument("--ref-pushes", type=int, default=24, help="pushes per step of the reference arm")
    ap.add_argument("--headline-only", action="store_true", help="skip variants, single kernels, e2e, CPU baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
