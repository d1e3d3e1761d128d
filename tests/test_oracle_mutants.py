"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the CPU checker's
source (on the CPU, in a temporary directory), builds it, and requires that at least one pin
of test_oracle_pins.PINS fails on it.  The unmodified checker passes them all."""
from __future__ import annotations

import os

import pytest

import oracle
from tests.test_oracle_pins import PINS

# (name, old text, new text, which occurrence to replace)
MUTANTS = [
    ("sign_of_delay_term", "T d = w[i] - snap[i];", "T d = snap[i] - w[i];", 0),
    ("compensation_subtracted", "T u = gi + c;", "T u = gi - c;", 0),
    ("delay_factor_dropped", "c = c * d;", "c = c;", 0),
    ("g_not_squared", "T c = lam * gg;", "T c = lam * gi;", 0),
    ("compensation_ignored", "T p = eta * u;", "T p = eta * gi;", 0),
    ("update_added", "w[i] = w[i] - p;", "w[i] = w[i] + p;", 0),
    ("ms_weight_mu_twice", "T b = omm * gg;", "T b = mu * gg;", 0),
    ("ms_uses_g_not_g2", "T b = omm * gg;", "T b = omm * gi;", 0),
    ("eps_dropped", "T s = v + eps;", "T s = v;", 0),
    ("eps_outside_root", "T r = root<T>(s);", "T r = root<T>(v) + eps;", 0),
    ("lambda_from_previous_ms", "T s = v + eps;", "T s = (a / mu) + eps;", 0),
    ("no_root", "T r = root<T>(s);", "T r = s;", 0),
    ("ms_not_stored", "ms[i] = v;", "", 0),
    ("ms_starts_at_one", "ms[i] = (T)0;", "ms[i] = (T)1;", 0),
    ("snapshot_of_worker_0", "const T* snap = wb + (uint64_t)m * n;", "const T* snap = wb;", 0),
    ("pull_writes_worker_0", "wb[(uint64_t)m * n + i] = w[i];", "wb[i] = w[i];", 1),
    ("init_skips_backups", "wb[(uint64_t)m * n + i] = w[i];", "wb[(uint64_t)m * n + i] = (T)0;", 0),
    ("pull_advances_t", "pull<T>(n, r.worker, w, wb);", "pull<T>(n, r.worker, w, wb); if (t) *t += 1;", 0),
    ("gradient_buffer_0", "grads + (uint64_t)r.grad_id * grad_stride", "grads", 0),
    ("record_eta_ignored", "r.eta < 0.0f ? default_eta : (T)r.eta", "default_eta", 0),
    ("bf16_widened_wrong", "(uint32_t)h << 16", "(uint32_t)h << 15", 0),
    ("momentum_decay_dropped", "T bv = beta * vel[i];", "T bv = vel[i];", 0),
    ("momentum_velocity_not_kept", "vel[i] = nv;", "", 0),
    ("momentum_step_ignores_velocity", "p = nv;", "", 0),
    ("momentum_adds_old_velocity_twice", "T nv = bv + p;", "T nv = bv + p + bv;", 0),
    ("one_minus_mu_is_one", "const T omm = (T)1 - mu;", "const T omm = (T)1;", 0),
]


def _replace_nth(text: str, old: str, new: str, nth: int) -> str:
    pos = -1
    for _ in range(nth + 1):
        pos = text.index(old, pos + 1)
    return text[:pos] + new + text[pos + len(old):]


def _failed_pins(L) -> list[str]:
    bad = []
    for pin in PINS:
        try:
            pin(L)
        except Exception:  # an assertion, or the mutant rejecting / corrupting its inputs
            bad.append(pin.__name__)
    return bad


def test_unmodified_checker_passes_every_pin(oracle_lib):
    assert _failed_pins(oracle_lib) == []


@pytest.mark.parametrize("name,old,new,nth", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, name, old, new, nth):
    with open(oracle.SRC) as f:
        src = f.read()
    mutated = _replace_nth(src, old, new, nth)
    assert mutated != src
    cpp = os.path.join(tmp_path, f"{name}.cpp")
    so = os.path.join(tmp_path, f"lib{name}.so")
    with open(cpp, "w") as f:
        f.write(mutated)
    L = oracle._bind(oracle.build(force=True, src=cpp, so=so))
    assert _failed_pins(L), f"no pin noticed the planted mistake '{name}'"
