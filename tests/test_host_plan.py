"""CPU tests of the library's host side: the shared object loads and exports
every symbol the header declares, and the host graph builder (levels, CSR in
level order, reachability relation, validation) is right. No GPU involved."""
from __future__ import annotations

import ctypes
import os
import re

import numpy as np
import pytest

import paper_1906_08879_b200 as placeto
from gen import configs, graphs
from tests.helpers import closure, random_dag, rng

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "placeto.h")).read()
    declared = set(re.findall(r"\b(placeto_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(placeto.binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(placeto.EXPORTS)


def test_status_strings():
    assert placeto.binding.status_string(0) == "ok"
    assert "DAG" in placeto.binding.status_string(2)
    assert placeto.binding.status_string(99) == "unknown status"


def _check_plan(n, src, dst):
    g = placeto.Graph(n, src, dst, host_only=True)
    view = g.host_view()
    info = g.info()
    edges = set(zip(map(int, src), map(int, dst)))
    assert info["n"] == n and info["n_edges"] == len(edges)
    par = [sorted(u for (u, v) in edges if v == w) for w in range(n)]
    chi = [sorted(v for (u, v) in edges if u == w) for w in range(n)]
    for name, nbrs in (("down", par), ("up", chi)):
        v = view[name]
        assert sorted(v["order"].tolist()) == list(range(n))
        level = np.empty(n, dtype=np.int64)
        for l in range(v["n_levels"]):
            seg = v["order"][v["level_ptr"][l]:v["level_ptr"][l + 1]]
            assert len(seg) > 0 and (np.diff(seg) > 0).all()
            level[seg] = l
        assert v["level_ptr"][0] == 0 and v["level_ptr"][-1] == n
        for p, node in enumerate(v["order"]):
            got = v["nbr"][v["nbr_ptr"][p]:v["nbr_ptr"][p + 1]].tolist()
            assert got == nbrs[node]
            # longest-path layering: one more than the deepest neighbour
            want = 1 + max(level[u] for u in nbrs[node]) if nbrs[node] else 0
            assert level[node] == want
    for name in ("down", "up"):
        _check_slots(view[name])
    assert info["n_levels_down"] == view["down"]["n_levels"] == graphs.depth(n, src, dst)
    assert info["n_levels_up"] == view["up"]["n_levels"] == info["n_levels_down"]
    R = closure(n, src, dst)
    rel = view["relation"]
    want = np.full((n, n), 2, dtype=np.uint8)
    want[R.T] = 0          # rel[c][u] = 0 when u reaches c
    want[R] = 1            # rel[c][u] = 1 when c reaches u
    np.fill_diagonal(want, 3)
    np.testing.assert_array_equal(rel, want)
    g.close()


def _check_slots(v):
    """Replays the level walk: every neighbour's slot must still hold that
    neighbour's message when it is read, and a level never writes a slot that
    the same level reads."""
    n = len(v["order"])
    holder = {}                                   # slot -> node whose message it holds
    consumers = np.zeros(n, dtype=bool)
    consumers[v["nbr"]] = True
    for l in range(v["n_levels"]):
        span = range(v["level_ptr"][l], v["level_ptr"][l + 1])
        read = set()
        for p in span:
            for e in range(v["nbr_ptr"][p], v["nbr_ptr"][p + 1]):
                s = v["nbr_slot"][e]
                assert 0 <= s < v["n_slots"] and holder[s] == v["nbr"][e]
                read.add(s)
        written = set()
        for p in span:
            s = v["own_slot"][p]
            node = v["order"][p]
            assert (s >= 0) == bool(consumers[node])
            if s >= 0:
                assert s < v["n_slots"] and s not in read and s not in written
                written.add(s)
                holder[s] = node
    assert v["n_slots"] <= max(1, int(consumers.sum()))


def test_plan_small_shapes():
    e = np.zeros(0, np.int32)
    _check_plan(1, e, e)                                       # single node
    _check_plan(5, e, e)                                       # isolated nodes
    _check_plan(6, np.arange(5), np.arange(1, 6))              # chain
    _check_plan(6, np.zeros(5, np.int32), np.arange(1, 6))     # star out
    _check_plan(6, np.arange(1, 6), np.zeros(5, np.int32))     # star in
    _check_plan(4, [0, 0, 1, 2, 0, 0], [1, 2, 3, 3, 1, 3])     # diamond + repeat + shortcut
    _check_plan(7, [0, 1, 3, 4], [1, 2, 4, 5])                 # two components + isolated


@pytest.mark.parametrize("seed", range(6))
def test_plan_random(seed):
    r = rng(100 + seed)
    n = int(r.integers(2, 40))
    src, dst = random_dag(r, n, float(r.uniform(0.05, 0.5)))
    _check_plan(n, src, dst)


@pytest.mark.parametrize("name", ["tiny", "inception", "nmt"])
def test_plan_configs(name):
    cfg = configs.make(name, B=1)
    _check_plan(cfg["n"], cfg["src"], cfg["dst"])


def test_plan_rejects_bad_graphs():
    def status(n, src, dst):
        with pytest.raises(placeto.PlacetoError) as e:
            placeto.Graph(n, src, dst, host_only=True)
        return e.value.status
    assert status(3, [0, 1, 2], [1, 2, 0]) == 2        # cycle
    assert status(3, [1], [1]) == 2                    # self-loop
    assert status(3, [0], [3]) == 2                    # id out of range
    assert status(3, [-1], [2]) == 2
    assert status(0, [], []) == 1                      # empty graph
    assert status(1 << 20, [], []) == 1                # beyond the node limit


def test_plan_at_the_node_limit():
    n = 16384                                           # PLACETO_MAX_NODES
    src = np.arange(n - 1, dtype=np.int32)
    g = placeto.Graph(n, src, src + 1, host_only=True)  # a chain: depth n, two alternating slots
    info = g.info()
    assert info["n_levels_down"] == n and info["max_level_width"] == 1
    view = g.host_view()
    assert view["down"]["n_slots"] == 2 and view["up"]["n_slots"] == 2
    rel = view["relation"]
    assert rel[0, n - 1] == 1 and rel[n - 1, 0] == 0 and rel[5, 5] == 3
    g.close()
    with pytest.raises(placeto.PlacetoError):
        placeto.Graph(n + 1, src, src + 1, host_only=True)


def test_workspace_bytes_on_host_graph():
    cfg = configs.make("tiny")
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"], host_only=True)

    class W:                                            # sizes only: no device needed
        pass
    w = W()
    w.c = placeto.binding._Weights()
    w.c.d, w.c.F, w.c.m = cfg["d"], cfg["F"], cfg["m"]
    n, B, d, F = cfg["n"], cfg["B"], cfg["d"], cfg["F"]
    embed = placeto.placeto_workspace_bytes(g, w, B, placeto.CALL_EMBED)
    assert embed >= 2 * n * B * d * 4
    fwd = placeto.placeto_workspace_bytes(g, w, B, placeto.CALL_FORWARD)
    assert fwd >= embed + n * B * (F + 2 * d) * 4
    host = placeto.placeto_workspace_bytes(g, w, B, placeto.CALL_FORWARD_HOST)
    assert host >= fwd + 2 * n * B
    assert placeto.placeto_workspace_bytes(g, w, 0, placeto.CALL_EMBED) == 0
    assert placeto.placeto_workspace_bytes(g, w, B, placeto.CALL_EMBED, flags=3) == 0   # two schedules
    # forward calls refuse a host-only graph before touching the device
    ws = np.zeros(16, dtype=np.uint8)
    rc = placeto.binding._lib.placeto_embed_forward(
        g.handle, ctypes.byref(w.c), None, ctypes.c_int32(B), None, None, None,
        ctypes.c_size_t(0), ctypes.c_uint32(0), None)
    assert rc == 1
    del ws
