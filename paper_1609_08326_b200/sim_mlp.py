"""Simulated asynchronous training on one GPU: M workers (Algorithm 1) against the CUDA server
(Algorithm 2), under a seeded event order.

    python -m paper_1609_08326_b200.sim_mlp [--pushes 2000] [--workers 8] [--eta 0.02]
    python -m paper_1609_08326_b200.sim_mlp --sweep          # the study of lambda_0 (supplementary material)

The model is a 2-layer MLP (784 -> 512 ReLU -> 10, fp32, 407,050 parameters) with the softmax
cross-entropy loss of Section 2 of the paper, on a synthetic 10-class Gaussian mixture (60,000
samples, class means ~ N(0,1), within-class std 2.0).  A worker that PUSHes computes its
mini-batch gradient at the snapshot it last pulled, i.e. at the server's own w_bak[m]; that is
the workers' side of the protocol and is done with plain torch matmuls here (TF32 off).  The
update itself - every pull and every push - goes through the dcasgd_* library calls.

Three runs share one gradient noise sequence: sequential SGD (tau = 0: pull right before every
push), ASGD (lambda = 0) and DC-ASGD-a.  `observer(t, m, g, srv)` is called after every push
(the tests hand each gradient to the CPU checker there and compare w step by step).

`--sweep` repeats the DC-ASGD-a run for several lambda_0 on a harder setting (more workers with
Zipf-distributed speeds, hence long delays, and a mixture whose classes overlap), the shape of
the paper's own study of lambda_0: a value that is too large hurts, a value that is too small
degenerates to ASGD (lambda_0 = 0 IS the ASGD trajectory, bit for bit).  A run can be stopped after
any push, saved with `Server.state_dict()` and continued by a new server (`state=`, `stop_after=`).
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as B
from . import synth

D_IN, D_HID, D_OUT = 784, 512, 10
N_PARAMS = D_IN * D_HID + D_HID + D_HID * D_OUT + D_OUT          # 407,050
N_SAMPLES, BATCH = 60_000, 128
STREAM_MEANS, STREAM_X, STREAM_Y, STREAM_BATCH = 0x2001, 0x2002, 0x2003, 0x2100


def make_data(seed: int, device, noise_std: float = 2.0, normalize: bool = False):
    """Gaussian mixture: x = mean[y] + noise_std * z; with `normalize`, divided by noise_std
    (unit-variance noise, class means pulled together: the classes overlap for a large noise_std)."""
    import torch
    means = synth.normal(D_OUT * D_IN, seed, STREAM_MEANS, 1.0).reshape(D_OUT, D_IN)
    y = (synth.u32(N_SAMPLES, seed, STREAM_Y).astype(np.uint64) * D_OUT >> 32).astype(np.int64)
    x = synth.normal(N_SAMPLES * D_IN, seed, STREAM_X, noise_std).reshape(N_SAMPLES, D_IN)
    x += means[y]
    if normalize:
        x *= np.float32(1.0 / noise_std)
    return torch.from_numpy(x).to(device), torch.from_numpy(y).to(device)


def init_params(seed: int) -> np.ndarray:
    """w_0: layer weights ~ N(0, 1/fan_in), biases 0, flat in the order W1, b1, W2, b2."""
    w = np.zeros(N_PARAMS, dtype=np.float32)
    w[: D_IN * D_HID] = synth.normal(D_IN * D_HID, seed, synth.STREAM_W0, D_IN ** -0.5)
    o = D_IN * D_HID + D_HID
    w[o: o + D_HID * D_OUT] = synth.normal(D_HID * D_OUT, seed, synth.STREAM_W0 + 1, D_HID ** -0.5)
    return w


def split(flat):
    o1 = D_IN * D_HID
    o2 = o1 + D_HID
    o3 = o2 + D_HID * D_OUT
    return flat[:o1].view(D_HID, D_IN), flat[o1:o2], flat[o2:o3].view(D_OUT, D_HID), flat[o3:]


def loss_and_grad(flat, x, y, g_out=None):
    """Mean softmax cross-entropy of the mini-batch and, if g_out is given, its gradient
    (mean over the batch) written flat into g_out."""
    import torch
    W1, b1, W2, b2 = split(flat)
    h = torch.relu(x @ W1.t() + b1)
    logits = h @ W2.t() + b2
    logp = torch.log_softmax(logits, dim=1)
    loss = -logp.gather(1, y[:, None]).mean()
    if g_out is not None:
        gW1, gb1, gW2, gb2 = split(g_out)
        dlogits = torch.exp(logp)
        dlogits.scatter_add_(1, y[:, None], torch.full((y.numel(), 1), -1.0, device=flat.device))
        dlogits /= y.numel()
        torch.mm(dlogits.t(), h, out=gW2)
        torch.sum(dlogits, dim=0, out=gb2)
        dh = dlogits @ W2
        dh *= (h > 0)
        torch.mm(dh.t(), x, out=gW1)
        torch.sum(dh, dim=0, out=gb1)
    return loss


def run(mode: str, pushes: int, M: int = 8, eta: float = 0.02, lam0: float = 2.0, mu: float = 0.95,
        eps: float = 1e-7, seed: int = 0, data=None, observer=None, eval_every: int = 50, device="cuda",
        order: int = synth.ORDER_UNIFORM, order_param: float = 0.0, stop_after: int | None = None,
        state: dict | None = None):
    """mode: 'sgd' (tau = 0), 'asgd' (lambda = 0), 'dcasgd-c' (constant lambda = lam0) or 'dcasgd-a'.
    Returns (server, loss curve, log).  `stop_after`: stop once that many pushes (counted from the
    start of the log) are applied.  `state`: a dictionary from `Server.state_dict()` of a run that
    was stopped that way; the run continues at the log record after its last push."""
    import torch
    torch.backends.cuda.matmul.allow_tf32 = False
    x_all, y_all = data if data is not None else make_data(seed, device)
    proto = synth.PROTO_TAU0 if mode == "sgd" else synth.PROTO_ASYNC
    ev = synth.event_log(M, pushes, order, proto, 1, eta, seed, order_param)
    adaptive = mode == "dcasgd-a"
    lam = lam0 if mode in ("dcasgd-a", "dcasgd-c") else 0.0
    srv = B.Server(init_params(seed) if state is None else None, M, adaptive, eta, lam, mu if adaptive else 0.0,
                   eps if adaptive else 0.0, device=device, state=state)
    picks = synth.u32(pushes * BATCH, seed, STREAM_BATCH).astype(np.uint64) * N_SAMPLES >> 32
    picks = torch.from_numpy(picks.astype(np.int64).reshape(pushes, BATCH)).to(device)
    g = torch.empty(N_PARAMS, dtype=torch.float32, device=device)
    eval_idx = torch.arange(0, N_SAMPLES, N_SAMPLES // 2048, device=device)[:2048]
    curve, t, first = [], 0, 0
    if state is not None:                                 # skip the records the saved run had already applied
        t = int(state["t"])
        push_rec = np.flatnonzero(ev["kind"] == synth.PUSH)
        first = int(push_rec[t - 1]) + 1 if t > 0 else 0
    for r in ev[first:]:
        if stop_after is not None and t >= stop_after:
            break
        m = int(r["worker"])
        if r["kind"] == synth.PULL:
            srv.pull(m)
            continue
        idx = picks[t]
        loss_and_grad(srv.w_bak[m], x_all[idx], y_all[idx], g)        # Algorithm 1: gradient at the pulled snapshot
        srv.push(m, g, float(r["eta"]))
        t += 1
        if observer is not None:
            observer(t, m, g, srv)
        if t % eval_every == 0 or t == pushes:
            curve.append((t, float(loss_and_grad(srv.w, x_all[eval_idx], y_all[eval_idx]))))
    return srv, curve, ev


SWEEP_LAMBDA0 = (0.0, 0.04, 0.5, 2.0, 8.0, 32.0)
SWEEP = dict(M=16, order=synth.ORDER_ZIPF, order_param=1.2, noise_std=14.0, eta=0.3, pushes=3000)


def sweep(pushes: int | None = None, seed: int = 0, lambdas=SWEEP_LAMBDA0, data=None, eval_every: int = 100, **override) -> dict:
    """DC-ASGD-a for several lambda_0 (and ASGD and sequential SGD beside them) on the hard
    setting SWEEP: 16 workers with Zipf(1.2) speeds (the slow ones push with delays of dozens of
    updates), overlapping classes.  Returns the loss curves on a fixed evaluation subset."""
    cfg = dict(SWEEP, **override)
    if pushes:
        cfg["pushes"] = pushes
    data = data if data is not None else make_data(seed, "cuda", cfg["noise_std"], normalize=True)
    common = dict(M=cfg["M"], eta=cfg["eta"], seed=seed, data=data, eval_every=eval_every)
    out = {"model": "mlp 784-512-10", "params": N_PARAMS, "setting": {k: v for k, v in cfg.items()}, "curves": {}}
    _, out["curves"]["sgd"], _ = run("sgd", cfg["pushes"], **common)
    _, out["curves"]["asgd"], ev = run("asgd", cfg["pushes"], order=cfg["order"], order_param=cfg["order_param"], **common)
    tau = synth.delays(ev, cfg["M"])
    out["delay"] = {"mean": float(tau.mean()), "p90": float(np.percentile(tau, 90)), "max": int(tau.max())}
    for lam0 in lambdas:
        _, curve, _ = run("dcasgd-a", cfg["pushes"], lam0=lam0, order=cfg["order"], order_param=cfg["order_param"], **common)
        out["curves"][f"dcasgd-a lambda0={lam0:g}"] = curve
    out["final_loss"] = {k: v[-1][1] for k, v in out["curves"].items()}
    out["mean_loss_last_quarter"] = {k: float(np.mean([l for _, l in v[-max(1, len(v) // 4):]])) for k, v in out["curves"].items()}
    return out


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--pushes", type=int, default=0)
    ap.add_argument("--workers", type=int, default=8)
    ap.add_argument("--eta", type=float, default=0.02)
    ap.add_argument("--lambda0", type=float, default=2.0)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--sweep", action="store_true", help="the lambda_0 study on the hard setting")
    ap.add_argument("--noise-std", type=float, default=0.0, help="sweep: within-class standard deviation")
    ap.add_argument("--sweep-eta", type=float, default=0.0)
    a = ap.parse_args()
    if a.sweep:
        over = {}
        if a.noise_std:
            over["noise_std"] = a.noise_std
        if a.sweep_eta:
            over["eta"] = a.sweep_eta
        print(json.dumps(sweep(a.pushes or None, a.seed, **over)))
        return
    pushes = a.pushes or 2000
    data = make_data(a.seed, "cuda")
    out = {"model": "mlp 784-512-10", "params": N_PARAMS, "workers": a.workers, "pushes": pushes, "eta": a.eta}
    for mode in ("sgd", "asgd", "dcasgd-a"):
        _, curve, _ = run(mode, pushes, a.workers, a.eta, a.lambda0, seed=a.seed, data=data)
        out[mode] = curve
    print(json.dumps(out))


if __name__ == "__main__":
    main()
