"""Pins of the CPU policy-gradient checker (oracle/gradient.py): its PyTorch
restatement of the forward must reproduce the C checker's log-probabilities,
and its gradient must match central finite differences of the C checker's
objective, weight by weight, on entries of every network; plus closed forms for
the last layer's bias and the entropy term."""
from __future__ import annotations

import copy

import numpy as np
import pytest
import torch

from gen import states
from oracle import gradient, oracle
from tests.helpers import random_dag, rng


def _case(seed, n=9, m=3, d=4, B=5, layers=2):
    r = rng(seed)
    src, dst = random_dag(r, n, 0.3)
    cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
    cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(r, n, m, B)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, layers, 0, 0.3)
    actions = r.integers(0, m, B)
    adv = r.normal(size=B)
    return cfg, actions, adv


def _objective_c(cfg, actions, adv, beta):
    p = oracle.forward(cfg)["probs"]
    logp = np.log(p)
    return float((adv * logp[np.arange(len(actions)), actions]).sum() - beta * (p * logp).sum())


@pytest.mark.parametrize("layers", [1, 2])
def test_restated_forward_reproduces_the_c_checker(layers):
    cfg, actions, adv = _case(3 + layers, layers=layers)
    logp = gradient.forward(cfg, gradient.tensors(cfg["weights"])).detach().numpy()
    np.testing.assert_allclose(np.exp(logp), oracle.forward(cfg)["probs"], rtol=0, atol=1e-12)


@pytest.mark.parametrize("beta", [0.0, 0.7])
def test_gradient_matches_finite_differences_of_the_c_checker(beta):
    cfg, actions, adv = _case(11)
    g = gradient.gradient(cfg, actions, adv, beta)
    assert abs(g["J"] - _objective_c(cfg, actions, adv, beta)) < 1e-10
    r = rng(5)
    eps = 1e-5
    checked = 0
    targets = [("f_down", None), ("g_down", None), ("f_up", None), ("g_up", None), ("head", None)]
    targets += [("l", i) for i in range(3)] + [("h", i) for i in range(3)]
    for name, idx in targets:
        net = cfg["weights"][name] if idx is None else cfg["weights"][name][idx]
        gnet = g[name] if idx is None else g[name][idx]
        for key in ("W1", "b1", "W2", "b2"):
            if net.get(key) is None:
                continue
            arr = net[key]
            for _ in range(2):
                pos = tuple(int(r.integers(0, s)) for s in arr.shape)
                keep = arr[pos]
                # the weights are float32 arrays: perturb in float32 and use the realised step
                arr[pos] = np.float32(keep + eps * max(1.0, abs(keep)) * 100)
                hi, up = float(arr[pos]), _objective_c(cfg, actions, adv, beta)
                arr[pos] = np.float32(keep - eps * max(1.0, abs(keep)) * 100)
                lo, down = float(arr[pos]), _objective_c(cfg, actions, adv, beta)
                arr[pos] = keep
                fd = (up - down) / (hi - lo)
                assert abs(fd - gnet[key][pos]) <= 2e-4 * max(1.0, abs(fd)), (name, idx, key, pos, fd, gnet[key][pos])
                checked += 1
    assert checked >= 40


def test_last_bias_and_entropy_closed_forms():
    cfg, actions, adv = _case(21)
    B, m = len(actions), cfg["m"]
    p = oracle.forward(cfg)["probs"]
    # d/d(head b2) of sum_b A_b log p_b[a_b] = sum_b A_b (onehot(a_b) - p_b)
    g0 = gradient.gradient(cfg, actions, adv, 0.0)
    onehot = np.eye(m)[actions]
    np.testing.assert_allclose(g0["head"]["b2"], (adv[:, None] * (onehot - p)).sum(axis=0), atol=1e-10)
    # entropy alone: dH/dlogit_k = -p_k (log p_k + H)
    ge = gradient.gradient(cfg, actions, np.zeros(B), 1.0)
    H = -(p * np.log(p)).sum(axis=1, keepdims=True)
    np.testing.assert_allclose(ge["head"]["b2"], (-p * (np.log(p) + H)).sum(axis=0), atol=1e-10)
    # linear in the advantages
    g2 = gradient.gradient(cfg, actions, 2 * adv, 0.0)
    np.testing.assert_allclose(g2["f_down"]["W1"], 2 * g0["f_down"]["W1"], rtol=1e-10, atol=1e-14)
