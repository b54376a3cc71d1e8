"""The five workload configurations: graph + raw states + weights per name.

Each configuration owns one ``Generator(PCG64(seed))``; the draw order is
graph (its own generator, same seed), then node costs, states, weights.
"""
from __future__ import annotations

import numpy as np

from . import graphs, states

# name -> (graph recipe, seed, m, d, B); F = m + 4
_CONFIGS = {
    "tiny": (graphs.layered_dag, 1, 2, 8, 16),
    "inception": (graphs.inception_shaped, 2, 4, 32, 256),
    "nmt": (graphs.nmt_shaped, 3, 4, 32, 256),
    "nasnet": (graphs.nasnet_shaped, 4, 8, 64, 512),
    # same recipe with the shorter op chains and two lanes per op (half the depth): timed beside "nasnet"
    "nasnet_wide": (graphs.nasnet_shaped_wide, 4, 8, 64, 512),
}

NAMES = ("tiny", "inception", "nmt", "nasnet", "sweep")


def _pack(name, n, src, dst, m, d, cost, nbytes, dev, cur, placed, weights):
    return {"name": name, "n": int(n), "src": src, "dst": dst, "m": m, "d": d,
            "F": m + 4, "B": int(dev.shape[0]), "cost": cost, "bytes": nbytes,
            "dev": dev, "cur": cur, "placed": placed, "weights": weights,
            "depth": graphs.depth(n, src, dst)}


def make(name: str, B: int | None = None, normalise: bool = False,
         bias_scale: float = 0.1):
    """Builds configuration `name` ("tiny", "inception", "nmt", "nasnet").

    `B` overrides the batch size (the draws of the first states do not depend
    on it only when it is left alone; parity cases that shrink the batch state
    so). `normalise` divides costs and byte counts by their means.
    """
    recipe, seed, m, d, B0 = _CONFIGS[name]
    B = B0 if B is None else B
    n, src, dst = recipe(seed)
    rng = np.random.Generator(np.random.PCG64(seed))
    cost, nbytes = states.node_costs(rng, n, normalise)
    dev, cur, placed = states.random_states(rng, n, m, B)
    weights = states.policy_weights(rng, d, m + 4, m, 2, 0, bias_scale)
    return _pack(name, n, src, dst, m, d, cost, nbytes, dev, cur, placed, weights)


def make_sweep(i: int, normalise: bool = False, count: int = 64):
    """Graph i (0..63) of the full-episode sweep with the n states of one
    episode: 8 devices, d = 32, B = n."""
    m, d = 8, 32
    n, src, dst = graphs.sweep_graph(i, count)
    rng = np.random.Generator(np.random.PCG64(1000 + i))
    cost, nbytes = states.node_costs(rng, n, normalise)
    dev, cur, placed = states.episode_states(rng, n, src, dst, m)
    weights = states.policy_weights(rng, d, m + 4, m, 2, 0, 0.1)
    return _pack("sweep%02d" % i, n, src, dst, m, d, cost, nbytes, dev, cur,
                 placed, weights)
