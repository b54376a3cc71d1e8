"""CPU checker for the "simple aggregator" policy of the paper's ablation
(Sec. 4.3, "Alternative policy architectures", variant 1). Test infrastructure
only: the CUDA library shares no code with it.

The paper: one feed-forward network aggregates all the node features of the
graph, and the result is fed to another feed-forward network with softmax
outputs. No message passing, no sets, no graph structure at all.

Readings (the paper gives no formula):
  - "aggregates all node features" is the sum over ALL nodes of a per-node
    network, squashed like the pooling summaries of Sec. 2.2 step 3:
        a = h( sum_{u in V} l(x_u) ),   l: F -> d,  h: d -> d;
    a sum because graphs differ in size; the current node is in the sum like
    every other node and is told apart by its is-current feature only;
  - the second network is the head: logits = head(a), head: d -> hidden -> m,
    probs = softmax(logits) (max-subtracted);
  - networks follow the one- or two-layer convention of the other checkers.
Plain fp64 numpy loops over states and nodes, ascending node id.
"""
from __future__ import annotations

import numpy as np


def _mlp(net, v):
    act = (lambda t: np.maximum(t, 0.0)) if net["act"] == 0 else (lambda t: t)
    y = v @ np.asarray(net["W1"], dtype=np.float64) + np.asarray(net["b1"], dtype=np.float64)
    if net["n_layers"] == 2:
        y = act(y)
        y = y @ np.asarray(net["W2"], dtype=np.float64) + np.asarray(net["b2"], dtype=np.float64)
    if net["final_act"]:
        y = act(y)
    return y


def simple_aggregator(X, weights):
    """X: [n][B][F] raw features; weights: {"l", "h", "head"} network dicts.
    Returns (logits [B][m], probs [B][m]) in fp64."""
    X = np.asarray(X, dtype=np.float64)
    n, B, _ = X.shape
    logits = []
    for b in range(B):
        s = None
        for u in range(n):
            y = _mlp(weights["l"], X[u, b])
            s = y if s is None else s + y
        logits.append(_mlp(weights["head"], _mlp(weights["h"], s)))
    logits = np.asarray(logits)
    e = np.exp(logits - logits.max(axis=1, keepdims=True))
    return logits, e / e.sum(axis=1, keepdims=True)
