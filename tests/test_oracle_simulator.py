"""Pins of the CPU runtime simulator (oracle/simulator.py) against timelines
that the execution model of the paper's Appendix A.5 fixes by hand: one device,
chains, independent chains, a fork-join with a transfer in each direction, a
bus that serialises two transfers, FIFO order on a device, and bounds and
closed forms on random graphs (critical path, device load, exact scaling).
"""
from __future__ import annotations

import numpy as np
import pytest

from gen import graphs
from oracle import simulator
from tests.helpers import random_dag, rng


def longest_path(n, src, dst, cost):
    order = graphs.topological_order(n, src, dst)
    par = [[] for _ in range(n)]
    for u, v in set(zip(map(int, src), map(int, dst))):
        par[v].append(u)
    finish = np.zeros(n)
    for v in order:
        finish[v] = cost[v] + max([finish[u] for u in par[v]], default=0.0)
    return float(finish.max())


def test_one_device_runs_everything_back_to_back():
    r = rng(1)
    src, dst = random_dag(r, 12, 0.3)
    cost = r.uniform(0.5, 2.0, 12).astype(np.float32)
    size = r.uniform(1, 9, 12).astype(np.float32)
    t = simulator.runtime(12, src, dst, cost, size, np.zeros(12, int), 1, 3.0)
    assert abs(t - float(np.sum(cost.astype(np.float64)))) < 1e-9


def test_chain_across_alternating_devices_pays_every_transfer():
    n = 7
    src, dst = np.arange(n - 1), np.arange(1, n)
    cost = np.arange(1, n + 1).astype(np.float32)
    size = (10 * np.arange(1, n + 1)).astype(np.float32)
    dev = np.arange(n) % 2
    t = simulator.runtime(n, src, dst, cost, size, dev, 2, 5.0)
    assert abs(t - (cost.sum() + size[:-1].sum() / 5.0)) < 1e-9
    # same device all along: no transfer at all
    assert abs(simulator.runtime(n, src, dst, cost, size, np.ones(n, int), 2, 5.0) - cost.sum()) < 1e-9


def test_independent_chains_on_their_own_devices_overlap():
    src = np.array([0, 1, 3, 4, 5]); dst = np.array([1, 2, 4, 5, 6])      # chains 0-1-2 and 3-4-5-6
    cost = np.array([1, 2, 3, 1, 1, 1, 1.5], dtype=np.float32)
    size = np.ones(7, dtype=np.float32)
    dev = np.array([0, 0, 0, 1, 1, 1, 1])
    assert simulator.runtime(7, src, dst, cost, size, dev, 2, 1.0) == 6.0
    assert simulator.runtime(7, src, dst, cost, size, np.zeros(7, int), 2, 1.0) == 10.5


def test_fork_join_timeline_by_hand():
    # a -> {b, c} -> d ; b on device 1, the rest on device 0; bandwidth 2
    src = np.array([0, 0, 1, 2]); dst = np.array([1, 2, 3, 3])
    cost = np.array([1.0, 4.0, 2.0, 1.0], dtype=np.float32)
    size = np.array([2.0, 6.0, 1.0, 1.0], dtype=np.float32)
    dev = np.array([0, 1, 0, 0])
    # a: 0..1; a's output to device 1: 1..2; b: 2..6; c on device 0: 1..3;
    # b's output to device 0: 6..9; d: 9..10
    assert simulator.runtime(4, src, dst, cost, size, dev, 2, 2.0) == 10.0
    # a faster link: b's output arrives at 6 + 0.75, d ends at 7.75
    assert simulator.runtime(4, src, dst, cost, size, dev, 2, 8.0) == 1 + 0.25 + 4 + 0.75 + 1


def test_bus_sends_one_tensor_at_a_time_and_once_per_device():
    # a on device 0 feeds b, c on device 1 and d on device 2
    src = np.array([0, 0, 0]); dst = np.array([1, 2, 3])
    cost = np.array([1.0, 1.0, 1.0, 5.0], dtype=np.float32)
    size = np.array([4.0, 1, 1, 1], dtype=np.float32)
    dev = np.array([0, 1, 1, 2])
    # to device 1: 1..3 (once, for b and c); to device 2: 3..5; b: 3..4, c: 4..5; d: 5..10
    assert simulator.runtime(4, src, dst, cost, size, dev, 3, 2.0) == 10.0
    # the other child order on the bus: d's device named first
    dev2 = np.array([0, 2, 1, 1])       # b on 2 (first child), c and d on 1
    cost2 = np.array([1.0, 5.0, 1.0, 1.0], dtype=np.float32)
    # to device 2: 1..3, b: 3..8; to device 1: 3..5, c: 5..6, d: 6..7
    assert simulator.runtime(4, src, dst, cost2, size, dev2, 3, 2.0) == 8.0


def test_device_queue_is_first_in_first_out():
    # roots 0 and 1 on device 0 (0 first); 2 depends on 1 and sits on device 1
    src = np.array([1]); dst = np.array([2])
    cost = np.array([5.0, 1.0, 1.0], dtype=np.float32)
    size = np.array([1.0, 2.0, 1.0], dtype=np.float32)
    dev = np.array([0, 0, 1])
    # 0: 0..5, 1: 5..6, transfer 6..8, 2: 8..9
    assert simulator.runtime(3, src, dst, cost, size, dev, 2, 1.0) == 9.0


@pytest.mark.parametrize("seed", range(5))
def test_bounds_and_closed_forms_on_random_graphs(seed):
    r = rng(40 + seed)
    n, m = 30, 4
    src, dst = random_dag(r, n, 0.12)
    cost = r.lognormal(0, 1, n).astype(np.float32)
    size = r.lognormal(2, 1, n).astype(np.float32)
    dev = r.integers(0, m, n)
    c64 = cost.astype(np.float64)
    t = simulator.runtime(n, src, dst, cost, size, dev, m, 10.0)
    crit = longest_path(n, src, dst, c64)
    load = max(c64[dev == d].sum() for d in range(m))
    assert t >= crit - 1e-9 and t >= load - 1e-9
    assert t <= c64.sum() + size.astype(np.float64).sum() * (m - 1) / 10.0 + 1e-9
    # a device per operation and an infinitely fast link: the critical path exactly
    free = simulator.runtime(n, src, dst, cost, size, np.arange(n), n, float("inf"))
    assert abs(free - crit) < 1e-9
    # times scale exactly with a power of two
    t2 = simulator.runtime(n, src, dst, 2 * cost, size, dev, m, 5.0)
    assert t2 == 2 * t
    # a faster link never makes a chain-free schedule of one device slower
    assert simulator.runtime(n, src, dst, cost, size, np.zeros(n, int), m, 1.0) == pytest.approx(c64.sum())


# ------------------------------------------------ peak memory and R(p) ----

def _sim(src, dst, cost, size, dev, m, bw=1.0):
    n = len(cost)
    return simulator.simulate(n, np.asarray(src), np.asarray(dst), np.asarray(cost, np.float32),
                              np.asarray(size, np.float32), dev, m, bw)


def test_memory_timelines_by_hand():
    """Appendix A.5: start and end of every operation plus the tensor sizes give
    the devices' peak memory. Timelines small enough to follow by eye."""
    # chain a -> b -> c on one device, sizes 10, 20, 5:
    # a runs: 10; b runs: 10 + 20 = 30; b done frees a's output: 20; c runs: 25; c done frees b's: 5
    r, peak = _sim([0, 1], [1, 2], [1, 1, 1], [10, 20, 5], [0, 0, 0], 1)
    assert r == 3.0 and peak.tolist() == [30.0]
    # a on device 0 feeds b on device 1: the receive buffer counts from the start of the transfer
    # device 0: 10 while a runs and until its output has left; device 1: 10, then 10 + 20 while b runs
    r, peak = _sim([0], [1], [1, 1], [10, 20], [0, 1], 2, bw=10.0)
    assert r == 3.0 and peak.tolist() == [10.0, 30.0]
    # fork a -> {b, c} on one device: a's output stays until BOTH children are done
    # a: 10; b: 30; b done: a still needed by c; c: 35; c done frees a's
    r, peak = _sim([0, 0], [1, 2], [1, 1, 1], [10, 20, 5], [0, 0, 0], 1)
    assert peak.tolist() == [35.0]
    # the same fork with c on device 1: device 0 holds a's output until b is done AND the copy has left
    # device 0: a 10, b +20 = 30; device 1: copy of a 10, c +5 = 15
    r, peak = _sim([0, 0], [1, 2], [1, 1, 1], [10, 20, 5], [0, 0, 1], 2, bw=10.0)
    assert peak.tolist() == [30.0, 15.0]
    # a -> {b on device 0, c on device 1}, b -> e on device 0, a slow link (the copy of a's output
    # is under way from t = 1 to t = 101): a's output stays at home while it is being sent, so e
    # runs on top of it. device 0: a 10, b 30, e 30 + 50 = 80; device 1: copy 10, c 15
    r, peak = _sim([0, 0, 1], [1, 2, 3], [1, 1, 1, 1], [10, 20, 5, 50], [0, 0, 1, 0], 2, bw=0.1)
    assert r == 102.0 and peak.tolist() == [80.0, 15.0]
    # outputs of operations without children are never released: three roots on one device pile up
    r, peak = _sim([], [], [1, 1, 1], [4, 5, 6], [0, 0, 0], 1)
    assert peak.tolist() == [15.0]


def test_memory_invariants_on_random_graphs():
    r = rng(77)
    for _ in range(6):
        n, m = 25, 3
        src, dst = random_dag(r, n, 0.15)
        cost = r.lognormal(0, 1, n).astype(np.float32)
        size = r.integers(1, 50, n).astype(np.float32)      # integers: sums are exact
        dev = r.integers(0, m, n)
        _, peak = simulator.simulate(n, src, dst, cost, size, dev, m, 7.0)
        chi, _ = simulator.children_lists(n, src, dst)
        for d in range(m):
            own = [v for v in range(n) if dev[v] == d]
            # a device holds at least its largest own output and all its childless outputs at the end
            if own:
                assert peak[d] >= max(size[v] for v in own)
                assert peak[d] >= sum(size[v] for v in own if not chi[v])
            # and never more than everything that is ever placed or copied there
            copies = sum(size[u] for u in range(n) if dev[u] != d and any(dev[c] == d for c in chi[u]))
            assert peak[d] <= sum(size[v] for v in own) + copies
        # one device, no transfers: the peak does not depend on the bandwidth
        a = simulator.simulate(n, src, dst, cost, size, np.zeros(n, int), 1, 1.0)[1]
        b = simulator.simulate(n, src, dst, cost, size, np.zeros(n, int), 1, 99.0)[1]
        assert a.tolist() == b.tolist()


def test_memory_penalised_runtime():
    """Appendix A.7: R(p) = r below the limit, r + c (m - M) above it."""
    assert simulator.penalised_runtime(3.0, 10.0, 10.7, 2.0) == 3.0
    assert simulator.penalised_runtime(3.0, 10.7, 10.7, 2.0) == 3.0
    assert simulator.penalised_runtime(3.0, 12.7, 10.7, 2.0) == 3.0 + 2.0 * 2.0
    src, dst = np.array([0, 0]), np.array([1, 2])
    devs = np.array([[0, 0, 0], [0, 0, 1]])
    r, peaks, pen = simulator.placements(3, src, dst, np.ones(3, np.float32), np.array([10, 20, 5], np.float32),
                                         devs, 2, 10.0, 32.0, 2.0)
    assert peaks.tolist() == [[35.0, 0.0], [30.0, 15.0]]
    assert pen[0] == r[0] + 2.0 * 3.0 and pen[1] == r[1]


@pytest.mark.parametrize("old,new", [
    ("        if any(dev[c] == d and not finished[c] for c in chi[u]):\n            return\n", ""),   # freed at the first child
    ("        hold(to, o)\n", ""),                                                                  # receive buffer not counted
    ("        if d == dev[u] and tr_left[u] > 0:\n            return\n", ""),                      # freed before it was sent
    ("return r if peak <= mem_limit else r + scale * (peak - mem_limit)",
     "return r if peak <= mem_limit else r - scale * (peak - mem_limit)"),                          # penalty sign
], ids=["freed at first child", "receive buffer dropped", "freed before sent", "penalty sign"])
def test_planted_memory_mistakes_are_caught(old, new, monkeypatch):
    import importlib.util, os, sys, tempfile
    path = simulator.__file__
    source = open(path).read()
    assert source.count(old) == 1
    with tempfile.TemporaryDirectory() as tmp:
        mut = os.path.join(tmp, "mutant_simulator.py")
        open(mut, "w").write(source.replace(old, new))
        spec = importlib.util.spec_from_file_location("mutant_simulator", mut)
        module = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(module)
    this = sys.modules[__name__]
    monkeypatch.setattr(this, "simulator", module)
    caught = False
    for pin in (test_memory_timelines_by_hand, test_memory_penalised_runtime, test_memory_invariants_on_random_graphs):
        try:
            pin()
        except AssertionError:
            caught = True
            break
    assert caught
