"""CPU checker of a placement episode (test infrastructure only, like the rest
of oracle/): the MDP of Sec. 2.1 of the Placeto paper driven by the policy of
Sec. 2.2, one step at a time, plain and slow.

Sec. 2.1: a state carries, per node, its device, a visited flag and a flag on
the one current node. At a step the agent picks a device for the current node;
the node is then marked visited and an unvisited node becomes current; after
|V| steps every node has been updated. The order of the visits is arbitrary in
the paper and an input here. All E episodes of a call share the graph, the
weights and the visiting order and differ in their initial devices and in the
random numbers that drive the sampling.

The policy forward of each step is oracle.forward in fp64. The discrete choice
(an argmax, or an inverse-CDF sample) is taken on the logits rounded to fp32
with fp32 arithmetic in index order, which is the precision and order the CUDA
library decides in. Beside each action the rollout reports how far that decision was
from flipping, so that a comparison can stop where rounding may legitimately
change the trajectory.
"""
from __future__ import annotations

import numpy as np

from . import oracle


def choose(logits64: np.ndarray, u=None):
    """Decision for one state. logits64: fp64 [m]. u: None for greedy, else a
    uniform number in [0, 1).

    Greedy: the largest logit, the lowest index among equals; margin = gap to
    the runner-up. Sampling: p = softmax (max-subtracted), the first index k
    with p_0 + .. + p_k > u (the last index if rounding leaves none); margin =
    distance from u to the nearest boundary of the chosen interval.
    Returns (action, log p[action], margin); log p from the fp64 logits.
    """
    l32 = logits64.astype(np.float32)
    m = len(l32)
    shifted = logits64 - logits64.max()
    logp_all = shifted - np.log(np.exp(shifted).sum())
    if u is None:
        a = 0
        for k in range(1, m):
            if l32[k] > l32[a]:
                a = k
        others = np.delete(logits64, a)
        margin = float(logits64[a] - others.max()) if m > 1 else np.inf
        return a, float(logp_all[a]), margin
    mx = np.float32(l32.max())
    e = np.exp((l32 - mx).astype(np.float32)).astype(np.float32)
    tot = np.float32(0)
    for k in range(m):
        tot = np.float32(tot + e[k])
    cum = np.float32(0)
    a = m - 1
    lo = np.float32(0)
    for k in range(m):
        lo = cum
        cum = np.float32(cum + np.float32(e[k] / tot))
        if cum > np.float32(u):
            a = k
            break
    hi = float(cum) if a < m - 1 else 1.0
    margin = min(float(u) - float(lo), hi - float(u))
    return a, float(logp_all[a]), margin


def rollout(cfg: dict, order, dev0, uniforms=None, threads=1):
    """Runs E episodes. cfg: n, src, dst, m, cost, bytes, weights (as in
    gen.configs). order: int [n], the node visited at step t. dev0: uint8
    [E][n] initial devices. uniforms: None (greedy) or float [E][n], the number
    that drives the choice of step t.

    Returns dict: actions int [E][n] (by step), logp [E][n] (by step), margin
    [E][n], dev uint8 [E][n] (final placement by node), logits [E][n][m] (by step).
    """
    n, m = cfg["n"], cfg["m"]
    order = np.asarray(order, dtype=np.int64)
    dev = np.array(dev0, dtype=np.uint8, copy=True)
    E = dev.shape[0]
    placed = np.zeros((E, n), dtype=np.uint8)
    actions = np.zeros((E, n), dtype=np.int64)
    logp = np.zeros((E, n))
    margin = np.zeros((E, n))
    all_logits = np.zeros((E, n, m))
    step_cfg = {k: cfg[k] for k in ("n", "src", "dst", "m", "cost", "bytes", "weights")}
    for t in range(n):
        v = int(order[t])
        step_cfg["dev"] = dev
        step_cfg["placed"] = placed
        step_cfg["cur"] = np.full(E, v, dtype=np.int32)
        logits = oracle.forward(step_cfg, threads=threads)["logits"]
        all_logits[:, t] = logits
        for e in range(E):
            u = None if uniforms is None else float(uniforms[e, t])
            a, lp, mg = choose(logits[e], u)
            actions[e, t], logp[e, t], margin[e, t] = a, lp, mg
            dev[e, v] = a           # the action: the current node's new device
            placed[e, v] = 1        # the transition: the node is visited
    return {"actions": actions, "logp": logp, "margin": margin, "dev": dev, "logits": all_logits}
