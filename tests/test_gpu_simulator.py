"""GPU parity of placeto_simulate_runtime against the CPU simulator: the
simulated run times are doubles produced by the same additions and divisions
in the same order, so they must be equal bit for bit."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs
from oracle import simulator
from tests.helpers import random_dag, rng

pytestmark = pytest.mark.gpu


def dev_t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_runtimes(n, src, dst, cost, size, devs, m, bw):
    g = placeto.Graph(n, src, dst)
    out = placeto.placeto_simulate_runtime(g, dev_t(cost), dev_t(size), dev_t(devs.astype(np.uint8)), m, bw)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("seed", range(4))
def test_random_graphs_bit_exact(seed):
    r = rng(70 + seed)
    n = int(r.integers(5, 60))
    m = int(r.integers(1, 7))
    src, dst = random_dag(r, n, float(r.uniform(0.05, 0.4)))
    cost = r.lognormal(0, 1, n).astype(np.float32)
    size = r.lognormal(3, 1.5, n).astype(np.float32)
    devs = r.integers(0, m, size=(37, n))
    bw = float(r.uniform(1, 50))
    got = gpu_runtimes(n, src, dst, cost, size, devs, m, bw)
    want = simulator.runtimes(n, src, dst, cost, size, devs, m, bw)
    np.testing.assert_array_equal(got, want)


def test_hand_timelines_and_ties():
    # fork-join with a transfer each way (see the CPU pins): 10.0 at bandwidth 2
    src = np.array([0, 0, 1, 2], np.int32); dst = np.array([1, 2, 3, 3], np.int32)
    cost = np.array([1.0, 4.0, 2.0, 1.0], np.float32)
    size = np.array([2.0, 6.0, 1.0, 1.0], np.float32)
    devs = np.array([[0, 1, 0, 0], [0, 0, 0, 0], [1, 1, 1, 1], [0, 1, 1, 0]])
    got = gpu_runtimes(4, src, dst, cost, size, devs, 2, 2.0)
    want = simulator.runtimes(4, src, dst, cost, size, devs, 2, 2.0)
    np.testing.assert_array_equal(got, want)
    assert got[0] == 10.0 and got[1] == 8.0 and got[2] == 8.0
    # integer costs and sizes: many events share a time stamp
    r = rng(5)
    n, m = 40, 3
    src, dst = random_dag(r, n, 0.15)
    cost = r.integers(1, 4, n).astype(np.float32)
    size = r.integers(1, 4, n).astype(np.float32)
    devs = r.integers(0, m, size=(64, n))
    np.testing.assert_array_equal(gpu_runtimes(n, src, dst, cost, size, devs, m, 1.0),
                                  simulator.runtimes(n, src, dst, cost, size, devs, m, 1.0))


@pytest.mark.parametrize("name,P", [("inception", 300), ("nmt", 64)])
def test_workload_graphs(name, P):
    cfg = configs.make(name, B=1)
    r = rng(9)
    n, m = cfg["n"], cfg["m"]
    devs = r.integers(0, m, size=(P, n))
    devs[0] = 0                                      # everything on one device
    got = gpu_runtimes(n, cfg["src"], cfg["dst"], cfg["cost"], cfg["bytes"], devs, m, 1e4)
    sel = np.arange(0, P, max(1, P // 24))
    want = simulator.runtimes(n, cfg["src"], cfg["dst"], cfg["cost"], cfg["bytes"], devs[sel], m, 1e4)
    np.testing.assert_array_equal(got[sel], want)
    assert abs(got[0] - cfg["cost"].astype(np.float64).sum()) < 1e-6 * got[0]


def test_errors_and_invalid_devices():
    r = rng(2)
    n, m = 10, 2
    src, dst = random_dag(r, n, 0.3)
    cost = np.ones(n, np.float32); size = np.ones(n, np.float32)
    devs = r.integers(0, m, size=(3, n))
    devs[1, 4] = 5                                   # a device that does not exist
    got = gpu_runtimes(n, src, dst, cost, size, devs, m, 1.0)
    assert np.isnan(got[1]) and np.isfinite(got[[0, 2]]).all()
    g = placeto.Graph(n, src, dst)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(placeto.PlacetoError) as e:
        placeto.placeto_simulate_runtime(g, dev_t(cost), dev_t(size), dev_t(devs.astype(np.uint8)), m, 1.0, ws=small)
    assert e.value.status == 3
    with pytest.raises(placeto.PlacetoError) as e:
        placeto.placeto_simulate_runtime(g, dev_t(cost), dev_t(size), dev_t(devs.astype(np.uint8)), m, 0.0)
    assert e.value.status == 1


def test_peak_memory_and_penalised_runtime_bit_exact():
    """placeto_simulate_placements against the CPU simulator: run time, per-device peak
    memory and R(p) (Appendix A.5, A.7) are doubles produced by the same operations in the
    same order."""
    for seed in range(4):
        r = rng(90 + seed)
        n = int(r.integers(5, 60))
        m = int(r.integers(1, 7))
        src, dst = random_dag(r, n, float(r.uniform(0.05, 0.4)))
        cost = r.lognormal(0, 1, n).astype(np.float32)
        size = r.lognormal(3, 1.5, n).astype(np.float32)
        devs = r.integers(0, m, size=(41, n))
        bw = float(r.uniform(1, 50))
        limit = float(np.percentile(size, 90)) * 2
        g = placeto.Graph(n, src, dst)
        rt, peak, pen = placeto.placeto_simulate_placements(g, dev_t(cost), dev_t(size), dev_t(devs.astype(np.uint8)),
                                                            m, bw, limit, 2.0)
        torch.cuda.synchronize()
        want_rt, want_peak, want_pen = simulator.placements(n, src, dst, cost, size, devs, m, bw, limit, 2.0)
        np.testing.assert_array_equal(rt.cpu().numpy(), want_rt)
        np.testing.assert_array_equal(peak.cpu().numpy(), want_peak)
        np.testing.assert_array_equal(pen.cpu().numpy(), want_pen)
        assert (pen.cpu().numpy() >= rt.cpu().numpy()).all() and (pen.cpu().numpy() > rt.cpu().numpy()).any()


def test_memory_timelines_by_hand_on_the_gpu():
    src = np.array([0, 0, 1], np.int32); dst = np.array([1, 2, 3], np.int32)
    cost = np.ones(4, np.float32); size = np.array([10, 20, 5, 50], np.float32)
    devs = np.array([[0, 0, 1, 0], [0, 0, 0, 0]], np.uint8)
    g = placeto.Graph(4, src, dst)
    rt, peak, pen = placeto.placeto_simulate_placements(g, dev_t(cost), dev_t(size), dev_t(devs), 2, 0.1, 75.0, 2.0)
    torch.cuda.synchronize()
    assert rt.cpu().tolist() == [102.0, 4.0]
    assert peak.cpu().tolist() == [[80.0, 15.0], [75.0, 0.0]]
    assert pen.cpu().tolist() == [102.0 + 2.0 * 5.0, 4.0]


def test_workload_graph_memory():
    cfg = configs.make("inception", B=1)
    r = rng(11)
    n, m = cfg["n"], cfg["m"]
    devs = r.integers(0, m, size=(64, n))
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    rt, peak, pen = placeto.placeto_simulate_placements(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]),
                                                        dev_t(devs.astype(np.uint8)), m, 1e4, 1e6, 2.0)
    torch.cuda.synchronize()
    sel = np.arange(0, 64, 8)
    want_rt, want_peak, want_pen = simulator.placements(n, cfg["src"], cfg["dst"], cfg["cost"], cfg["bytes"],
                                                        devs[sel], m, 1e4, 1e6, 2.0)
    np.testing.assert_array_equal(rt.cpu().numpy()[sel], want_rt)
    np.testing.assert_array_equal(peak.cpu().numpy()[sel], want_peak)
    np.testing.assert_array_equal(pen.cpu().numpy()[sel], want_pen)
