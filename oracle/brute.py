"""Exact brute-force evaluation of the policy on very small DAGs (test
infrastructure only).

Un-memoised recursion written directly from the definitions of Sec. 2.2 of
the paper, in exact rational arithmetic (``fractions.Fraction``), meant for
graphs of at most ~8 nodes with small-integer weights and features. It pins
the C checker: the two share no code and no data structures (this one works
on Python sets built from the edge list and never computes a topological
order or a level).
"""
from __future__ import annotations

from fractions import Fraction


def _frac(v):
    """Exact rational value of a Python or numpy number."""
    return v if isinstance(v, Fraction) else Fraction(float(v))


def _act(v, act):
    return v if (act == 1 or v > 0) else Fraction(0)


def _layer(W, b, v):
    return [sum((_frac(W[k][j]) * v[k] for k in range(len(v))), _frac(b[j]))
            for j in range(len(b))]


def mlp(net, v):
    """One or two feed-forward layers (Appendix A.7)."""
    y = _layer(net["W1"], net["b1"], v)
    if net["n_layers"] == 2:
        y = [_act(t, net["act"]) for t in y]
        y = _layer(net["W2"], net["b2"], y)
    if net["final_act"]:
        y = [_act(t, net["act"]) for t in y]
    return y


class Brute:
    def __init__(self, n, edges, weights):
        self.n = n
        self.edges = set((int(u), int(v)) for u, v in edges)
        self.w = weights

    def parents(self, v):
        return sorted(u for (u, t) in self.edges if t == v)

    def children(self, v):
        return sorted(t for (u, t) in self.edges if u == v)

    def h(self, v, x, down):
        """Embedding of v in one direction (Sec. 2.2 step 2): g of the sum of
        f([h_u || x_u]) over parents (down) or children (up); recursion ends
        at nodes without such neighbours."""
        f = self.w["f_down" if down else "f_up"]
        g = self.w["g_down" if down else "g_up"]
        d = self.w["d"]
        s = [Fraction(0)] * d
        for u in (self.parents(v) if down else self.children(v)):
            msg = mlp(f, self.h(u, x, down) + list(x[u]))
            s = [a + b for a, b in zip(s, msg)]
        return mlp(g, s)

    def can_reach(self, a, b):
        """True if a directed path of length >= 1 leads from a to b."""
        return any(t == b or self.can_reach(t, b) for t in self.children(a))

    def logits(self, x, c):
        """Pooling over the three sets of Sec. 2.2 step 3 and the head's
        pre-softmax outputs for current node c. x: per-node feature lists."""
        d = self.w["d"]
        emb = lambda u: self.h(u, x, True) + self.h(u, x, False) + list(x[u])
        sums = [[Fraction(0)] * d for _ in range(3)]
        for u in range(self.n):
            if u == c:
                continue
            i = 0 if self.can_reach(u, c) else (1 if self.can_reach(c, u) else 2)
            y = mlp(self.w["l"][i], emb(u))
            sums[i] = [a + b for a, b in zip(sums[i], y)]
        z = emb(c)
        for i in range(3):
            z = z + mlp(self.w["h"][i], sums[i])
        return mlp(self.w["head"], z)


def features(m, cost, nbytes, dev, cur, placed):
    """[cost, bytes, one-hot device, is-current, is-placed] per node for one
    state (Sec. 2.2 step 1)."""
    out = []
    for v in range(len(cost)):
        onehot = [Fraction(1 if int(dev[v]) == k else 0) for k in range(m)]
        out.append([_frac(cost[v]), _frac(nbytes[v])] + onehot
                   + [Fraction(1 if v == cur else 0), Fraction(1 if placed[v] else 0)])
    return out
