"""Child process of test_gpu_checked_build.py: runs with DCASGD_CHECKED_BUILD=1, i.e. against the
library compiled with -DDCASGD_DEBUG_CHECKS, whose kernels compare every global address with the
buffers of the call.  Replays a subset of the parity cases and prints the status word."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_1609_08326_b200 import binding as B  # noqa: E402
from paper_1609_08326_b200 import synth  # noqa: E402
from tests import gpu_util as U  # noqa: E402

assert os.environ.get("DCASGD_CHECKED_BUILD") == "1"
status = torch.zeros(1, dtype=torch.int32, device="cuda")
B.dcasgd_debug_checks(None, status)                       # servers created from here on report into it


def workload(n, adaptive, bf16, M=6, pushes=60, G=8, seed=1):
    return synth.Workload(name="t", n=n, M=M, pushes=pushes, adaptive=adaptive, bf16_grad=bf16, eta=0.1,
                          lam=2.0 if adaptive else 0.04, mu=0.95 if adaptive else 0.0, eps=1e-7 if adaptive else 0.0,
                          num_grads=G, nseg=3 if n >= 30 else 1, sigma_lo_exp=-4, sigma_hi_exp=-1, seed=seed)


mode = sys.argv[1]
if mode == "parity":
    cases = 0
    for vecs in ("1", "2"):
        os.environ["DCASGD_REPLAY_VECS"] = vecs
        for n in (1, 5, 1023, 1025, 2050, 50_001):
            for adaptive, bf16 in ((False, False), (True, False), (False, True), (True, True)):
                for beta in (None, 0.9):
                    wl = workload(n, adaptive, bf16, seed=n % 7)
                    ev, w0, pool = wl.log(), wl.w0(), U.host_pool(wl)
                    dpool = U.to_device(pool)
                    out_w = torch.empty(n, dtype=torch.float32, device="cuda")
                    for K in (1, 8, 1000):
                        gpu, cpu = U.gpu_server(wl, w0, beta=beta), U.cpu_server(wl, w0, beta=beta)
                        gpu.pull(1, out_w)
                        gpu.push(1, dpool[2], 0.05)
                        cpu.pull(1)
                        cpu.push(1, pool[2, :n], np.float32(0.05))
                        gpu.apply_log(ev, dpool, K)
                        cpu.replay(ev, pool[:, :n])
                        U.assert_state_equal(gpu, cpu)
                        gpu.close()
                        cases += 1
    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.dcasgd_check_adaptive_lambda(2.0, 1.0, 4.0, counter)
    torch.cuda.synchronize()
    print(f"CHECKED parity cases={cases} status={int(status.item())} lambda_mismatches={int(counter.item())}", flush=True)
elif mode == "selftest":
    # The access TABLE is made 16 bytes shorter than the buffers (DCASGD_CHECKED_SHRINK=16, set by
    # the parent): the kernels' own last vector then counts as out of range, is skipped and
    # reported.  The buffers themselves are whole, so nothing invalid is touched.
    assert os.environ.get("DCASGD_CHECKED_SHRINK") == "16"
    n = 4096
    wl = workload(n, True, False)
    w0, pool = wl.w0(), U.host_pool(wl)
    dpool = U.to_device(pool)
    gpu = U.gpu_server(wl, w0)                            # Initialize: the last vector of every array is skipped
    torch.cuda.synchronize()
    after_init = int(status.item())
    gpu.w_bak_buf.fill_(7.0)
    status.zero_()
    gpu.pull(wl.M - 1)                                    # the last slab ends where the (shortened) table ends
    torch.cuda.synchronize()
    after_pull = int(status.item())
    slab = gpu.w_bak[wl.M - 1].cpu().numpy()
    skipped = bool(np.all(slab[-4:] == 7.0)) and bool(np.array_equal(slab[:-4], gpu.w.cpu().numpy()[:-4]))
    status.zero_()
    gpu.push(0, dpool[0])
    torch.cuda.synchronize()
    after_push = int(status.item())
    print(f"CHECKED selftest init={after_init} pull={after_pull} push={after_push} skipped={int(skipped)}", flush=True)
