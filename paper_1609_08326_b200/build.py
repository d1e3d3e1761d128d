"""Builds the native parts of the package in-tree.

    python -m paper_1609_08326_b200.build          # everything
    python -m paper_1609_08326_b200.build synth    # only the input generator
    python -m paper_1609_08326_b200.build lib      # only the CUDA server library
    python -m paper_1609_08326_b200.build checked  # only its bounds-checked twin

Outputs (git-ignored shared objects next to their sources):
    synth/libdcasgd_synth.so   g++,  seeded input generator (host only)
    csrc/libdcasgd.so          nvcc, sm_100a, the C-ABI server library declared in include/dcasgd.h
    csrc/libdcasgd_checked.so  the same sources with -DDCASGD_DEBUG_CHECKS (bounds-checked kernels; tests only)
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)

SYNTH_SRC = os.path.join(PKG, "synth", "synth.cpp")
SYNTH_SO = os.path.join(PKG, "synth", "libdcasgd_synth.so")

LIB_SRCS = [os.path.join(PKG, "csrc", f) for f in ("dcasgd.cu", "window_compiler.cpp")]
LIB_HDRS = [os.path.join(PKG, "csrc", "window_compiler.h"),
            os.path.join(PKG, "csrc", "kernels.cuh"),
            os.path.join(ROOT, "include", "dcasgd.h")]
LIB_SO = os.path.join(PKG, "csrc", "libdcasgd.so")
LIB_CHECKED_SO = os.path.join(PKG, "csrc", "libdcasgd_checked.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    # every product rounds on its own (no a*b+c contraction): the kernels also spell each
    # operation with a round-to-nearest intrinsic, this flag covers the rest of the file
    "--fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC,-O2,-Wall",
    "-shared",
]


def _stale(target: str, sources: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources if os.path.exists(s))


def _run(cmd: list[str]) -> None:
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        sys.stderr.write(" ".join(cmd) + "\n" + proc.stdout + proc.stderr)
        raise RuntimeError(f"build step failed: {cmd[0]} (exit {proc.returncode})")
    if proc.stderr.strip():
        sys.stderr.write(proc.stderr)


def build_synth(force: bool = False) -> str:
    if force or _stale(SYNTH_SO, [SYNTH_SRC]):
        _run(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-Wall",
              "-o", SYNTH_SO, SYNTH_SRC])
    return SYNTH_SO


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the server library cannot be built")
    return cand


def build_lib(force: bool = False, verbose_ptxas: bool = False, debug_checks: bool = False) -> str:
    """debug_checks: the checked build (libdcasgd_checked.so) whose kernels compare every global
    address with the buffers of the call, skip what lies outside and report it in a status word."""
    so = LIB_CHECKED_SO if debug_checks else LIB_SO
    if force or _stale(so, LIB_SRCS + LIB_HDRS + [os.path.abspath(__file__)]):
        cmd = [nvcc_path(), *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"),
               "-I", os.path.join(PKG, "csrc")]
        if debug_checks:
            cmd += ["-DDCASGD_DEBUG_CHECKS"]
        if verbose_ptxas:
            cmd += ["-Xptxas", "-v"]
        cmd += ["-o", so, *LIB_SRCS]
        _run(cmd)
    return so


def build_all(force: bool = False) -> None:
    build_synth(force)
    build_lib(force)
    build_lib(force, debug_checks=True)


if __name__ == "__main__":
    what = sys.argv[1] if len(sys.argv) > 1 else "all"
    force = "--force" in sys.argv
    if what == "synth":
        print(build_synth(force))
    elif what == "lib":
        print(build_lib(force, verbose_ptxas="-v" in sys.argv))
    elif what == "checked":
        print(build_lib(force, verbose_ptxas="-v" in sys.argv, debug_checks=True))
    else:
        build_all(force)
        print(SYNTH_SO)
        print(LIB_SO)
