"""Seeded placement states and policy weights (raw inputs only).

A placement state (Sec. 2.1 of the paper) is, per node: the op cost, the
output size, the device the node currently sits on, a visited ("placed") flag
and a flag on the one current node. This module draws those raw quantities and
the network weights; turning them into the feature tensor and everything after
it is the method's arithmetic and lives elsewhere (CPU checker and CUDA library
each have their own).
"""
from __future__ import annotations

import numpy as np

from .graphs import topological_order


def node_costs(rng: np.random.Generator, n: int, normalise: bool = False):
    """cost ~ lognormal(0, 1) (ms), bytes ~ lognormal(10, 2); fp32.

    With `normalise` each vector is divided by its mean (a scale-free variant
    used beside the raw one: the raw byte counts reach 1e7 and push every
    activation to that scale).
    """
    cost = rng.lognormal(0.0, 1.0, size=n)
    nbytes = rng.lognormal(10.0, 2.0, size=n)
    if normalise:
        cost = cost / cost.mean()
        nbytes = nbytes / nbytes.mean()
    return cost.astype(np.float32), nbytes.astype(np.float32)


def random_states(rng: np.random.Generator, n: int, m: int, B: int):
    """B independent states: device uniform over m per node, one uniform
    current node per state, placed flag Bernoulli(0.5) for every node."""
    dev = rng.integers(0, m, size=(B, n)).astype(np.uint8)
    cur = rng.integers(0, n, size=B).astype(np.int32)
    placed = (rng.random(size=(B, n)) < 0.5).astype(np.uint8)
    return dev, cur, placed


def episode_states(rng: np.random.Generator, n: int, src, dst, m: int):
    """All n states of one placement episode that visits nodes in topological
    order: in state t the t-th node is current, the nodes before it are placed
    on uniform random devices, the rest (current included) are unplaced on
    device 0."""
    order = topological_order(n, src, dst)
    chosen = rng.integers(0, m, size=n).astype(np.uint8)   # device picked at step t
    dev = np.zeros((n, n), dtype=np.uint8)
    placed = np.zeros((n, n), dtype=np.uint8)
    for t in range(n):
        done = order[:t]
        dev[t, done] = chosen[:t]
        placed[t, done] = 1
    cur = order.astype(np.int32).copy()
    return dev, cur, placed


def _xavier(rng, fan_in: int, fan_out: int):
    a = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-a, a, size=(fan_in, fan_out)).astype(np.float32)


def _bias(rng, size: int, scale: float):
    return rng.uniform(-scale, scale, size=size).astype(np.float32)


def mlp_weights(rng, in_dim: int, hidden_dim: int, out_dim: int, n_layers: int,
                act: int = 0, final_act: int = 1, bias_scale: float = 0.1):
    """One feed-forward net as a dict: W row-major [in][out], Xavier-uniform;
    biases uniform in +-bias_scale. act: 0 relu, 1 identity. final_act: 1 if
    the activation also follows the last layer."""
    net = {"n_layers": n_layers, "in_dim": in_dim,
           "hidden_dim": hidden_dim if n_layers == 2 else out_dim,
           "out_dim": out_dim, "act": act, "final_act": final_act}
    if n_layers == 1:
        net["W1"] = _xavier(rng, in_dim, out_dim)
        net["b1"] = _bias(rng, out_dim, bias_scale)
        net["W2"] = None
        net["b2"] = None
    else:
        net["W1"] = _xavier(rng, in_dim, hidden_dim)
        net["b1"] = _bias(rng, hidden_dim, bias_scale)
        net["W2"] = _xavier(rng, hidden_dim, out_dim)
        net["b2"] = _bias(rng, out_dim, bias_scale)
    return net


def policy_weights(rng, d: int, F: int, m: int, mp_layers: int = 2,
                   act: int = 0, bias_scale: float = 0.1):
    """All networks of the policy, drawn in a fixed order.

    f: (d+F) -> d and g: d -> d per direction with `mp_layers` layers (the
    workload configurations use 2; the paper's Appendix A.7 uses 1);
    l_i: (2d+F) -> d and h_i: d -> d, one layer each, for the parent, child
    and parallel groups; head: (5d+F) -> (5d+F) -> m with a linear output.
    """
    w = {"d": d, "F": F, "m": m}
    for name in ("down", "up"):
        w["f_" + name] = mlp_weights(rng, d + F, d, d, mp_layers, act, 1, bias_scale)
        w["g_" + name] = mlp_weights(rng, d, d, d, mp_layers, act, 1, bias_scale)
    w["l"] = [mlp_weights(rng, 2 * d + F, 0, d, 1, act, 1, bias_scale) for _ in range(3)]
    w["h"] = [mlp_weights(rng, d, 0, d, 1, act, 1, bias_scale) for _ in range(3)]
    z = 5 * d + F
    w["head"] = mlp_weights(rng, z, z, m, 2, act, 0, bias_scale)
    return w
