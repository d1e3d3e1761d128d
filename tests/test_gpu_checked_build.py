"""The bounds-checked build of the library (-DDCASGD_DEBUG_CHECKS) stands in for a memory
checker: each kernel compares every global address it uses with the buffers of the call, skips
what lies outside and sets a bit in a status word.  A subset of the parity cases must run under
it with status 0; and with the access table deliberately made 16 bytes shorter than the (whole)
buffers, the kernels' last vectors must be reported and skipped - without any invalid access."""
from __future__ import annotations

import os
import re
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHILD = os.path.join(ROOT, "tests", "checked_build_child.py")


def run_child(mode: str, **env) -> str:
    from paper_1609_08326_b200 import build
    build.build_lib(debug_checks=True)
    e = dict(os.environ, DCASGD_CHECKED_BUILD="1", **env)
    e.pop("DCASGD_REPLAY_VECS", None)
    out = subprocess.run([sys.executable, CHILD, mode], capture_output=True, text=True, timeout=900, cwd=ROOT, env=e)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("CHECKED")]
    assert len(lines) == 1, out.stdout
    return lines[0]


def test_parity_subset_runs_clean_under_the_checked_build():
    line = run_child("parity")
    m = re.match(r"CHECKED parity cases=(\d+) status=(\d+) lambda_mismatches=(\d+)", line)
    assert m, line
    assert int(m.group(1)) == 2 * 6 * 4 * 2 * 3
    assert int(m.group(2)) == 0, "a kernel touched memory outside the buffers of its call"
    assert int(m.group(3)) == 0


def test_the_checker_reports_and_skips_when_the_table_is_short():
    line = run_child("selftest", DCASGD_CHECKED_SHRINK="16")
    m = re.match(r"CHECKED selftest init=(\d+) pull=(\d+) push=(\d+) skipped=(\d)", line)
    assert m, line
    init, pull, push, skipped = (int(x) for x in m.groups())
    assert init & 1 and init & 2          # last vector of w read and of w_bak / ms written: both refused
    assert pull == 3                      # bad read (w) and bad write (last slab of w_bak), nothing misaligned
    assert push & 1 and push & 2
    assert skipped == 1                   # the refused store did not happen; everything else did


def test_normal_build_has_no_checks():
    from paper_1609_08326_b200 import binding as B
    if os.environ.get("DCASGD_CHECKED_BUILD") == "1":
        pytest.skip("running against the checked build")
    with pytest.raises(B.DcasgdError) as e:
        B.dcasgd_debug_checks(None, None)
    assert e.value.status == B.EINVAL
