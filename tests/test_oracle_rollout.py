"""Pins of the CPU episode checker (oracle/rollout.py) against what the MDP of
Sec. 2.1 and elementary probability fix, independent of the checker itself:
a policy whose logits do not depend on the state (closed form for every action
and log-probability), the bookkeeping of the transition rebuilt from the
returned actions, a one-node graph, and the decision rule on hand-made logits.
"""
from __future__ import annotations

import numpy as np
import pytest

from gen import graphs, states
from oracle import oracle, rollout
from tests.helpers import random_dag, rng


def _case(seed, n=9, m=3, d=4, E=4, p=0.3):
    r = rng(seed)
    src, dst = random_dag(r, n, p)
    cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.1)
    order = graphs.topological_order(n, src, dst)
    dev0 = r.integers(0, m, size=(E, n)).astype(np.uint8)
    uni = r.random(size=(E, n))
    return cfg, order, dev0, uni


def test_decision_rule_on_hand_made_logits():
    # greedy: largest logit, lowest index among equals, margin = gap to the runner-up
    a, lp, mg = rollout.choose(np.array([1.0, 3.0, 3.0, 0.5]))
    assert a == 1 and mg == 0.0
    a, lp, mg = rollout.choose(np.array([0.0, np.log(3.0)]))
    assert a == 1 and abs(lp - np.log(0.75)) < 1e-12 and abs(mg - np.log(3.0)) < 1e-12
    # sampling: p = (0.25, 0.75); u below 0.25 picks 0, above picks 1
    lg = np.array([0.0, np.log(3.0)])
    a, lp, mg = rollout.choose(lg, 0.2)
    assert a == 0 and abs(lp - np.log(0.25)) < 1e-12 and abs(mg - 0.05) < 1e-6
    a, lp, mg = rollout.choose(lg, 0.9)
    assert a == 1 and abs(lp - np.log(0.75)) < 1e-12 and abs(mg - 0.1) < 1e-6
    # one device: always that device, probability one
    a, lp, mg = rollout.choose(np.array([-7.0]), 0.999)
    assert a == 0 and lp == 0.0


@pytest.mark.parametrize("greedy", [True, False])
def test_state_independent_policy_has_a_closed_form(greedy):
    """Head with zero weights: logits = the output bias for every state, so every
    action is the argmax of the bias (greedy) or the inverse CDF of softmax(bias)
    at the given uniform number, and log p follows."""
    cfg, order, dev0, uni = _case(3, m=4)
    head = cfg["weights"]["head"]
    head["W1"][:] = 0
    head["W2"][:] = 0
    bias = np.array([0.3, -1.0, 1.2, 0.1], dtype=np.float32)
    head["b2"][:] = bias
    out = rollout.rollout(cfg, order, dev0, None if greedy else uni)
    p = np.exp(bias.astype(np.float64))
    p /= p.sum()
    if greedy:
        want = np.full(dev0.shape, 2)
    else:
        want = np.minimum(np.searchsorted(np.cumsum(p), uni, side="right"), 3)
    np.testing.assert_array_equal(out["actions"], want)
    np.testing.assert_allclose(out["logp"], np.log(p)[want], atol=1e-6)
    # every node was visited once and carries the device chosen at its step
    np.testing.assert_array_equal(out["dev"][:, order], want)


def test_transition_bookkeeping_rebuilt_from_the_actions():
    """State t rebuilt independently from the returned actions (nodes visited
    before t carry their chosen device and the visited flag, the others their
    initial device; the t-th node of the order is current and not yet visited)
    must reproduce the logits the rollout saw at step t."""
    cfg, order, dev0, uni = _case(5, n=8, E=3)
    out = rollout.rollout(cfg, order, dev0, uni)
    n = cfg["n"]
    for t in (0, 1, n // 2, n - 1):
        dev = dev0.copy()
        placed = np.zeros_like(dev0)
        for s in range(t):
            dev[:, order[s]] = out["actions"][:, s]
            placed[:, order[s]] = 1
        c = dict(cfg)
        c.update(dev=dev, placed=placed, cur=np.full(len(dev0), order[t], dtype=np.int32))
        np.testing.assert_allclose(oracle.forward(c)["logits"], out["logits"][:, t], rtol=0, atol=1e-12)
    # a different visiting order changes the trajectory's states but still visits every node once
    rev = order[::-1].copy()
    out2 = rollout.rollout(cfg, rev, dev0, uni)
    np.testing.assert_array_equal(out2["dev"][:, rev], out2["actions"])
    assert (out2["actions"] >= 0).all() and (out2["actions"] < cfg["m"]).all()


def test_single_node_graph_is_one_policy_evaluation():
    r = rng(9)
    m, d = 3, 4
    cfg = {"n": 1, "src": np.zeros(0, np.int32), "dst": np.zeros(0, np.int32), "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, 1, normalise=True)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.1)
    dev0 = np.array([[0], [1], [2]], dtype=np.uint8)
    out = rollout.rollout(cfg, [0], dev0, None)
    c = dict(cfg)
    c.update(dev=dev0, placed=np.zeros_like(dev0), cur=np.zeros(3, np.int32))
    ref = oracle.forward(c)
    np.testing.assert_array_equal(out["actions"][:, 0], ref["logits"].argmax(axis=1))
    np.testing.assert_allclose(out["logp"][:, 0], np.log(ref["probs"].max(axis=1)), atol=1e-12)


def test_episodes_are_independent():
    cfg, order, dev0, uni = _case(7, E=5)
    full = rollout.rollout(cfg, order, dev0, uni)
    one = rollout.rollout(cfg, order, dev0[2:3], uni[2:3])
    np.testing.assert_array_equal(full["actions"][2], one["actions"][0])
    np.testing.assert_allclose(full["logp"][2], one["logp"][0], atol=1e-12)
