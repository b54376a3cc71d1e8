"""CPU checker of the policy gradient (test infrastructure only).

Appendix A.1 of the Placeto paper updates the parameters with
    sum_i grad_theta log pi(a_i | s_i) * (return_i - baseline_i)
(REINFORCE with a baseline), and Appendix A.7 adds an entropy term to the loss
to encourage exploration. For a batch of B states with their chosen actions
a_b, advantages A_b (return minus baseline, an input here) and an entropy
factor beta, this module returns the gradient, with respect to every weight
and bias of the policy, of
    J = sum_b A_b log pi(a_b | s_b) + beta sum_b H(pi(. | s_b)),
    H(p) = - sum_k p_k log p_k.

The policy forward is restated with plain PyTorch CPU operations in fp64 (the
same steps as oracle/placeto_oracle.c, which it must reproduce: a pin) and the
gradient comes from reverse-mode differentiation of that restatement; a second
pin compares it with finite differences of the C checker's log-probabilities.
"""
from __future__ import annotations

import numpy as np
import torch

from . import oracle

NETS = ("f_down", "g_down", "f_up", "g_up", "head")
SETS = ("l", "h")


def _topological(n, src, dst):
    par = [set() for _ in range(n)]
    chi = [set() for _ in range(n)]
    for u, v in zip(map(int, src), map(int, dst)):
        par[v].add(u)
        chi[u].add(v)
    indeg = [len(p) for p in par]
    order = [v for v in range(n) if indeg[v] == 0]
    for u in order:
        for v in sorted(chi[u]):
            indeg[v] -= 1
            if indeg[v] == 0:
                order.append(v)
    return order, [sorted(p) for p in par], [sorted(c) for c in chi]


def tensors(weights):
    """fp64 leaf tensors (requires_grad) for every array of the weight dict."""
    def net(w):
        t = {}
        for k in ("W1", "b1", "W2", "b2"):
            if w.get(k) is not None:
                t[k] = torch.tensor(np.asarray(w[k], dtype=np.float64), requires_grad=True)
        return t
    out = {k: net(weights[k]) for k in NETS}
    for k in SETS:
        out[k] = [net(w) for w in weights[k]]
    return out


def _act(v, a):
    return torch.relu(v) if a == 0 else v


def _mlp(w, t, v):
    y = v @ t["W1"] + t["b1"]
    if w["n_layers"] == 2:
        y = _act(y, w["act"]) @ t["W2"] + t["b2"]
    if w["final_act"]:
        y = _act(y, w["act"])
    return y


def forward(cfg, t):
    """log-softmax of the device logits, [B][m], as a differentiable fp64 tensor."""
    n, m, d = cfg["n"], cfg["m"], cfg["d"]
    W = cfg["weights"]
    X = torch.tensor(oracle.features(n, m, cfg["cost"], cfg["bytes"], cfg["dev"], cfg["cur"], cfg["placed"]))
    B = X.shape[1]
    order, par, chi = _topological(n, cfg["src"], cfg["dst"])

    def sweep(nodes, nbrs, f, g):
        H = [None] * n
        for v in nodes:
            s = torch.zeros((B, d), dtype=torch.float64)
            for u in nbrs[v]:
                s = s + _mlp(W[f], t[f], torch.cat([H[u], X[u]], dim=1))
            H[v] = _mlp(W[g], t[g], s)
        return H

    Hd = sweep(order, par, "f_down", "g_down")
    Hu = sweep(order[::-1], chi, "f_up", "g_up")
    E = torch.stack([torch.cat([Hd[u], Hu[u], X[u]], dim=1) for u in range(n)])     # [n][B][2d+F]
    cur = np.asarray(cfg["cur"], dtype=np.int64)
    mask = np.zeros((3, n, B))
    for b in range(B):
        group, _ = oracle.groups(n, cfg["src"], cfg["dst"], int(cur[b]))     # 0 / 1 / 2, 3 = the node itself
        for i in range(3):
            mask[i, :, b] = group == i
    mask = torch.tensor(mask)
    parts = [E[cur, torch.arange(B)]]
    for i in range(3):
        y = _mlp(W["l"][i], t["l"][i], E)                                           # [n][B][d]
        s = (y * mask[i][:, :, None]).sum(dim=0)
        parts.append(_mlp(W["h"][i], t["h"][i], s))
    logits = _mlp(W["head"], t["head"], torch.cat(parts, dim=1))
    return torch.log_softmax(logits, dim=1)


def objective(logp, actions, advantages, beta):
    B = logp.shape[0]
    chosen = logp[torch.arange(B), torch.tensor(np.asarray(actions, dtype=np.int64))]
    entropy = -(logp.exp() * logp).sum(dim=1)
    return (torch.tensor(np.asarray(advantages, dtype=np.float64)) * chosen).sum() + beta * entropy.sum()


def gradient(cfg, actions, advantages, beta=0.0):
    """Gradient of J with respect to every weight array: a dict shaped like the
    weight dict ({net: {W1, b1, W2, b2}}, lists for l and h) of fp64 arrays,
    plus "J" (the objective) and "logp"."""
    t = tensors(cfg["weights"])
    logp = forward(cfg, t)
    J = objective(logp, actions, advantages, beta)
    J.backward()
    def grads(net):
        # an array the objective does not depend on (f on a graph without edges) has no .grad: zero
        return {k: (v.grad.numpy().copy() if v.grad is not None else np.zeros(tuple(v.shape)))
                for k, v in net.items()}
    out = {k: grads(t[k]) for k in NETS}
    for k in SETS:
        out[k] = [grads(x) for x in t[k]]
    out["J"] = float(J.detach())
    out["logp"] = logp.detach().numpy()
    return out
