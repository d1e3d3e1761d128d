"""The C-ABI library without a GPU: it loads, exports every function the header declares, and
rejects bad arguments on the host before touching CUDA.  No compute call is made here."""
from __future__ import annotations

import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_1609_08326_b200 import binding as B
from paper_1609_08326_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dcasgd.h")


def declared_functions() -> list[str]:
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dcasgd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = B.lib()
    names = declared_functions()
    assert set(names) == set(B.SYMBOLS), "binding.SYMBOLS and include/dcasgd.h disagree"
    for name in names:
        assert getattr(L, name) is not None
    assert B.dcasgd_version() == 0x00010000
    assert B.status_string(B.ELOG) == "DCASGD_ELOG"


def test_struct_layouts_match_the_header():
    assert C.sizeof(B.Config) == 96
    assert B.Config.flags.offset == 36 and B.Config.w.offset == 40 and B.Config.w_bak_stride.offset == 56 and B.Config.ms.offset == 64 and B.Config.stream.offset == 72
    assert B.Config.v.offset == 80 and B.Config.beta.offset == 88 and B.Config.reserved.offset == 92
    assert synth.EVENT_DTYPE.itemsize == 16
    words = 6 + 3 * B.MAX_WINDOW_PUSHES + (B.MAX_WINDOW_PUSHES + 1) + (B.MAX_WINDOW_PUSHES + 2) + B.MAX_WINDOW_STORES
    assert C.sizeof(B.WindowProgram) == 4 * words
    hdr = open(HEADER).read()
    for name, val in (("PUSHES", B.MAX_WINDOW_PUSHES), ("STORES", B.MAX_WINDOW_STORES), ("SLOTS", B.MAX_WINDOW_SLOTS)):
        assert re.search(rf"#define DCASGD_MAX_WINDOW_{name} {val}\b", hdr)


def _create(**kw):
    # fake but well-formed addresses: validation must fail before any of them is dereferenced
    args = dict(n=1000, num_workers=4, variant=B.ADAPTIVE, grad_dtype=B.F32, eta=0.1, lam=2.0, mu=0.95,
                eps=1e-7, flags=0, w=0x10000, w_bak=0x20000, w_bak_stride=1000, ms=0x40000, stream=None)
    args.update(kw)
    return B.dcasgd_create(**args)


@pytest.mark.parametrize("kw,status", [
    (dict(num_workers=0), B.EINVAL), (dict(num_workers=70000), B.EINVAL),
    (dict(variant=2), B.EINVAL), (dict(grad_dtype=2), B.EINVAL), (dict(flags=2), B.EINVAL),
    (dict(beta=0.9), B.EINVAL), (dict(v=0x50000, beta=1.0), B.EINVAL), (dict(v=0x50000, beta=-0.5), B.EINVAL),
    (dict(v=0x50004, beta=0.9), B.EALIGN), (dict(v=0x10010, beta=0.9), B.EINVAL),       # v inside w
    (dict(eta=float("nan")), B.EINVAL), (dict(lam=float("inf")), B.EINVAL),
    (dict(mu=1.0), B.EINVAL), (dict(mu=-0.1), B.EINVAL), (dict(eps=-1e-7), B.EINVAL),
    (dict(ms=None), B.EINVAL), (dict(variant=B.CONST), B.EINVAL),          # ms given to the constant variant
    (dict(w=None), B.EINVAL), (dict(w_bak=None), B.EINVAL),
    (dict(w_bak_stride=999), B.EINVAL), (dict(w_bak_stride=1002), B.EALIGN),
    (dict(w=0x10004), B.EALIGN), (dict(w_bak=0x20008), B.EALIGN), (dict(ms=0x40001), B.EALIGN),
    (dict(ms=0x10100), B.EINVAL),                                         # ms inside w
    (dict(w_bak=0x10000 + 4000 - 16), B.EINVAL),                          # w_bak starts inside w
    (dict(w=0x20000 + 3 * 4000), B.EINVAL),                               # w inside the last backup slab
])
def test_create_rejects_bad_configs_on_the_host(kw, status):
    with pytest.raises(B.DcasgdError) as e:
        _create(**kw)
    assert e.value.status == status, e.value
    assert e.value.message


def test_null_handles_and_null_outputs():
    L = B.lib()
    assert L.dcasgd_destroy(None) == B.OK
    assert L.dcasgd_create(None, None) == B.EINVAL
    assert L.dcasgd_get_step(None, None) == B.EINVAL
    assert L.dcasgd_set_step(None, 3) == B.EINVAL
    assert L.dcasgd_get_launch_count(None, None) == B.EINVAL
    for call in (lambda: L.dcasgd_pull(None, 0, None), lambda: L.dcasgd_push(None, 0, None, C.c_float(0.1)),
                 lambda: L.dcasgd_apply_log(None, None, 0, None, 0, 0, 1)):
        assert call() == B.EINVAL
        assert "NULL" in B.last_error()


def test_valid_config_without_a_gpu_reports_a_cuda_error_not_a_crash():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(B.DcasgdError) as e:
        _create()
    assert e.value.status == B.ECUDA
