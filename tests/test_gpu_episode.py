"""GPU parity of placeto_episode_rollout against the CPU episode checker.

An episode feeds every discrete choice back into the next state, so one choice
that rounding flips changes everything after it. The comparison is therefore
exact (integer actions, the final placement) up to, and excluding, the first
step of an episode at which the checker's own decision was within MARGIN of
flipping (top-2 logit gap for greedy steps, distance of the uniform number from
the boundaries of the chosen probability interval for sampled ones); from there
on that episode is left out. The cases are chosen so that most episodes are
decisive to the end, and the test asserts that. Log-probabilities of the compared
steps agree within the logit tolerance of the parity tests.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs, graphs, states
from oracle import rollout
from tests.helpers import random_dag, rng

pytestmark = pytest.mark.gpu

MARGIN_LOGIT = 1e-3      # greedy: minimum top-2 gap, relative to max(1, |logits|_inf)
MARGIN_PROB = 1e-4       # sampled: minimum distance of u from an interval boundary


def dev_t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_gpu(cfg, order, dev0, uniforms, flags=0):
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    dev = dev_t(dev0)
    uni = None if uniforms is None else dev_t(uniforms.astype(np.float32))
    dev, actions, logp = placeto.placeto_episode_rollout(
        g, w, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(np.asarray(order, np.int32)), dev, uni,
        flags=flags)
    torch.cuda.synchronize()
    launches = placeto.placeto_last_launch_count()
    return dev.cpu().numpy(), actions.cpu().numpy(), logp.cpu().numpy(), launches


def compare(cfg, order, dev0, uniforms, got, min_full):
    dev, actions, logp, _ = got
    uni32 = None if uniforms is None else uniforms.astype(np.float32).astype(np.float64)
    ref = rollout.rollout(cfg, order, dev0, uni32, threads=8)
    E, n = dev0.shape
    scale = np.maximum(1.0, np.abs(ref["logits"]).max(axis=2))
    decisive = ref["margin"] > (MARGIN_LOGIT * scale if uniforms is None else MARGIN_PROB)
    full = 0
    for e in range(E):
        bad = np.flatnonzero(~decisive[e])
        upto = int(bad[0]) if len(bad) else n
        np.testing.assert_array_equal(actions[e, :upto], ref["actions"][e, :upto])
        np.testing.assert_allclose(logp[e, :upto], ref["logp"][e, :upto], atol=2e-4, rtol=2e-4)
        if upto == n:
            full += 1
            np.testing.assert_array_equal(dev[e], ref["dev"][e])
    assert full >= min_full, "only %d of %d episodes decisive to the end" % (full, E)
    # whatever the trajectory: every node carries the device chosen at its step
    np.testing.assert_array_equal(dev[:, np.asarray(order)], actions)
    assert (actions < cfg["m"]).all() and np.isfinite(logp).all() and (logp <= 0).all()


def small_case(seed, n, m, d, E, p=0.2):
    r = rng(seed)
    src, dst = random_dag(r, n, p)
    cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.1)
    order = graphs.topological_order(n, src, dst)
    dev0 = r.integers(0, m, size=(E, n)).astype(np.uint8)
    uni = r.random(size=(E, n))
    return cfg, order, dev0, uni


@pytest.mark.parametrize("sampled", [False, True])
@pytest.mark.parametrize("d,m,flags", [(32, 4, 0), (32, 4, placeto.PLACETO_TENSOR), (32, 3, 0), (8, 3, 0), (64, 8, 0)])
def test_small_graphs(d, m, flags, sampled):
    """d = 32 with F a multiple of 4 runs on compact states (one byte per node and episode, no
    feature tensor, the transition inside the head kernel: three kernels per step); the other
    cases, and d = 32 on the tensor kernel, keep the feature tensor and patch it (four)."""
    cfg, order, dev0, uni = small_case(100 * d + m, n=24, m=m, d=d, E=12)
    uniforms = uni if sampled else None
    got = run_gpu(cfg, order, dev0, uniforms, flags)
    compare(cfg, order, dev0, uniforms, got, min_full=9)
    compact = d == 32 and m == 4 and flags == 0
    assert got[3] == (24 * 3 + 2 if compact else 24 * 4 + 2)


def test_compact_states_with_initial_devices_beyond_the_device_count():
    """An initial placement may name devices the policy does not know (their one-hot is all
    zero); nodes keep them until visited. E = 70 episodes: several per block in every kernel."""
    cfg, order, dev0, uni = small_case(77, n=20, m=4, d=32, E=70)
    dev0[:, ::3] = 200
    dev0[:, 1::5] = 63
    got = run_gpu(cfg, order, dev0, uni)
    compare(cfg, order, dev0, uni, got, min_full=50)
    assert got[3] == 20 * 3 + 2


def test_reverse_order_and_single_episode():
    cfg, order, dev0, uni = small_case(5, n=16, m=4, d=32, E=1)
    order = order[::-1].copy()
    got = run_gpu(cfg, order, dev0, uni)
    compare(cfg, order, dev0, uni, got, min_full=0)


def test_one_node_graph():
    r = rng(3)
    m, d = 4, 32
    e = np.zeros(0, np.int32)
    cfg = {"n": 1, "src": e, "dst": e, "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, 1, normalise=True)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.1)
    dev0 = np.array([[0], [1], [2], [3], [0]], dtype=np.uint8)
    got = run_gpu(cfg, [0], dev0, None)
    compare(cfg, [0], dev0, None, got, min_full=4)


def test_inception_shaped_graph_sampled_episodes():
    """The Inception-shaped workload, 8 sampled episodes of 318 steps each."""
    cfg = configs.make("inception", B=1, normalise=True)
    r = rng(17)
    n, m = cfg["n"], cfg["m"]
    order = graphs.topological_order(n, cfg["src"], cfg["dst"])
    dev0 = np.zeros((8, n), dtype=np.uint8)           # everything starts on device 0
    uni = r.random(size=(8, n))
    got = run_gpu(cfg, order, dev0, uni)
    compare(cfg, order, dev0, uni, got, min_full=5)


def test_same_inputs_same_episode_and_argument_errors():
    cfg, order, dev0, uni = small_case(8, n=12, m=3, d=32, E=5)
    a = run_gpu(cfg, order, dev0, uni)
    b = run_gpu(cfg, order, dev0, uni)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[2], b[2])
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(placeto.PlacetoError) as err:
        placeto.placeto_episode_rollout(g, w, dev_t(cfg["cost"]), dev_t(cfg["bytes"]),
                                        dev_t(np.asarray(order, np.int32)), dev_t(dev0), ws=small)
    assert err.value.status == 3          # workspace too small: nothing launched
