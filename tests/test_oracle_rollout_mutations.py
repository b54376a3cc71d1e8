"""The pins of the episode checker must bite: each planted mistake in a copy
of oracle/rollout.py has to fail at least one test of test_oracle_rollout.py.
The mistakes live in the checker, on the CPU, only.
"""
from __future__ import annotations

import importlib.util
import os
import sys

import pytest

from oracle import rollout
from tests import test_oracle_rollout as pins

SRC = rollout.__file__

MUTATIONS = [
    ("ties go to the highest device", "if l32[k] > l32[a]:", "if l32[k] >= l32[a]:"),
    ("interval closed on the wrong side", "if cum > np.float32(u):", "if cum >= np.float32(1) or cum > np.float32(u) + np.float32(0.5):"),
    ("node marked visited before it is evaluated", "        step_cfg[\"placed\"] = placed\n",
     "        placed[:, v] = 1\n        step_cfg[\"placed\"] = placed\n"),
    ("action written to the step index, not the node", "            dev[e, v] = a ", "            dev[e, t] = a "),
    ("current node is the previous one", "np.full(E, v, dtype=np.int32)", "np.full(E, int(order[max(t - 1, 0)]), dtype=np.int32)"),
    ("log-probability of the wrong device", "return a, float(logp_all[a]), margin\n    mx =", "return a, float(logp_all[0]), margin\n    mx ="),
    ("episodes share one uniform number", "float(uniforms[e, t])", "float(uniforms[0, t])"),
    ("softmax without the max subtraction and without normalising", "cum = np.float32(cum + np.float32(e[k] / tot))", "cum = np.float32(cum + e[k])"),
]

PINS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]


def _run_pins(mod):
    """Runs every pin against `mod`; returns the names of those that fail."""
    failed = []
    saved = pins.rollout
    pins.rollout = mod
    try:
        for fn in PINS:
            params = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
            calls = [()] if not params else [(v,) for v in params[0].args[1]]
            for args in calls:
                try:
                    fn(*args)
                except Exception:          # an assertion or any error the mistake provokes
                    failed.append(fn.__name__)
                    break
    finally:
        pins.rollout = saved
    return failed


def _load(text, name):
    path = os.path.join(os.path.dirname(SRC), "_mutant_%s.py" % name)
    with open(path, "w") as f:
        f.write(text)
    try:
        spec = importlib.util.spec_from_file_location("oracle._mutant_%s" % name, path)
        mod = importlib.util.module_from_spec(spec)
        sys.modules[spec.name] = mod
        spec.loader.exec_module(mod)
        return mod
    finally:
        os.remove(path)


def test_the_unmodified_checker_passes_every_pin():
    assert _run_pins(rollout) == []


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_fails_a_pin(name, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation target not found exactly once: %r" % old
    mod = _load(text.replace(old, new), "".join(c if c.isalnum() else "_" for c in name)[:30])
    assert _run_pins(mod), "no pin noticed: " + name
