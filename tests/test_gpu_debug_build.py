"""The index-checking build of the library (-DPLACETO_DEBUG, libplaceto_debug.so):
the stand-in for a memory checker. Its kernels test the schedule records, slot,
node and state indices they stage and report a violation through the call's
status record; no access is made with a bad index and nothing traps.

The binding loads one library per process, so the checks run in a child
process with PLACETO_LIBRARY=debug.
"""
from __future__ import annotations

import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent('''
    import numpy as np, torch
    import paper_1906_08879_b200 as placeto
    from gen import configs, graphs, states
    from oracle import oracle
    assert placeto.binding.LIB_PATH.endswith("libplaceto_debug.so")
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()

    def run(cfg, flags):
        g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
        w = placeto.Weights(cfg["weights"])
        B = cfg["dev"].shape[0]
        ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD, flags)
        logits, _ = placeto.placeto_policy_forward(g, w, t(cfg["cost"]), t(cfg["bytes"]), t(cfg["dev"]), t(cfg["cur"]),
                                                   t(cfg["placed"]), ws=ws, flags=flags)
        status = placeto.placeto_last_status(g, ws)
        return g, w, ws, logits, status

    # every specialised kernel on a case with several states per block: no index out of range
    cases = {}
    for d, m, flags in ((32, 4, 0), (32, 4, placeto.PLACETO_TENSOR), (64, 8, 0), (64, 8, placeto.PLACETO_FMA_ONLY),
                        (64, 8, placeto.PLACETO_TCGEN05), (64, 8, placeto.PLACETO_TENSOR), (8, 2, 0)):
        rng = np.random.Generator(np.random.PCG64(d + flags))
        n, src, dst = graphs.layered_dag(seed=5, levels=12, width=5)
        cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4, "B": 200}
        cfg["cost"], cfg["bytes"] = states.node_costs(rng, n, True)
        cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(rng, n, m, 200)
        cfg["weights"] = states.policy_weights(rng, d, m + 4, m, 2, 0, 0.1)
        g, w, ws, logits, status = run(cfg, flags)
        assert status == 0, (d, flags, status)
        ref = oracle.forward(cfg, threads=4)["logits"]
        err = np.abs(logits.cpu().numpy() - ref).max() / np.abs(ref).max()
        assert err < 2e-5, (d, flags, err)
        cases[(d, flags)] = cfg

    # a current node outside [0, n): the release build answers NaN for that state (documented);
    # the debug build also reports the index, and the other states are untouched
    for d in (32, 64):
        cfg = cases[(d, 0)]
        cfg["cur"] = cfg["cur"].copy()
        cfg["cur"][3] = cfg["n"] + 5
        g, w, ws, logits, status = run(cfg, 0)
        assert status == 1, (d, status)
        assert torch.isnan(logits[3]).all() and torch.isfinite(logits[:3]).all() and torch.isfinite(logits[4:]).all()
    print("debug build ok")
''')


def test_index_checking_build_is_clean_on_valid_inputs_and_reports_a_bad_index():
    # incremental: a no-op when libplaceto_debug.so is newer than every source
    subprocess.run([sys.executable, os.path.join(ROOT, "paper_1906_08879_b200", "build.py"), "--debug"], check=True)
    env = dict(os.environ, PLACETO_LIBRARY="debug", PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "debug build ok" in out.stdout
