"""Seeded synthetic computation DAGs shaped like the paper's workloads.

The paper's own graphs (Inception-V3, NMT, NASNet and the ENAS-generated
cifar10 / ptb / nmt families, Sec. 3 and Appendix A.2-A.3) are TensorFlow graphs
that are not available; these recipes imitate their size and structure only
(chains of multi-branch blocks, an unrolled encoder-decoder grid with
attention, stacks of NAS cells, random conv / recurrent cells).

Every recipe draws from ``numpy.random.Generator(PCG64(seed))`` in a fixed
order and returns an edge list ``(n, src, dst)`` with ``src[i] -> dst[i]``.
This module holds graph construction only: none of the policy's arithmetic.
"""
from __future__ import annotations

import numpy as np


class _Builder:
    """Accumulates nodes and directed edges u -> v."""

    def __init__(self) -> None:
        self.n = 0
        self.src: list[int] = []
        self.dst: list[int] = []

    def node(self, *parents: int) -> int:
        v = self.n
        self.n += 1
        for u in parents:
            self.edge(u, v)
        return v

    def edge(self, u: int, v: int) -> None:
        self.src.append(int(u))
        self.dst.append(int(v))

    def chain(self, start: int, length: int) -> int:
        """Appends `length` nodes in a chain below `start`; returns the last."""
        cur = start
        for _ in range(length):
            cur = self.node(cur)
        return cur

    def done(self):
        return (self.n, np.asarray(self.src, dtype=np.int32),
                np.asarray(self.dst, dtype=np.int32))


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def layered_dag(seed: int = 1, levels: int = 8, width: int = 4):
    """Random layered DAG: `levels` x `width` nodes, ids level-major.

    Each node outside the last level draws an out-degree in {1,2,3} and that
    many distinct targets among the nodes of the next one or two levels. Every
    node below the first level is then guaranteed at least one parent (a
    uniform node of the level above is added when it drew none).
    """
    rng = _rng(seed)
    b = _Builder()
    ids = [[b.node() for _ in range(width)] for _ in range(levels)]
    has_parent = np.zeros(b.n, dtype=bool)
    for lv in range(levels - 1):
        cand = list(ids[lv + 1]) + (list(ids[lv + 2]) if lv + 2 < levels else [])
        for u in ids[lv]:
            deg = int(rng.integers(1, 4))
            deg = min(deg, len(cand))
            for v in rng.choice(len(cand), size=deg, replace=False):
                b.edge(u, cand[int(v)])
                has_parent[cand[int(v)]] = True
    for lv in range(1, levels):
        for v in ids[lv]:
            if not has_parent[v]:
                b.edge(ids[lv - 1][int(rng.integers(0, width))], v)
    return b.done()


def inception_shaped(seed: int = 2, stem: int = 20, modules: int = 11,
                     branches: int = 4):
    """A stem chain followed by multi-branch modules joined by concat nodes.

    Each module fans out of the previous join into `branches` parallel
    branches of 1-4 units; a unit is a conv -> bn or conv -> bn -> act chain
    (2 or 3 nodes, drawn per unit), which brings the total near 300 nodes.
    """
    rng = _rng(seed)
    b = _Builder()
    join = b.node()
    join = b.chain(join, stem - 1)
    for _ in range(modules):
        ends = []
        for _ in range(branches):
            units = int(rng.integers(1, 5))
            cur = join
            for _ in range(units):
                cur = b.chain(cur, int(rng.integers(2, 4)))
            ends.append(cur)
        join = b.node(*ends)
    return b.done()


def nmt_shaped(seed: int = 3, steps: int = 40, enc_layers: int = 2,
               dec_layers: int = 2):
    """Encoder-decoder LSTM grid unrolled `steps` timesteps, with attention.

    A cell at (t, layer) is six nodes: four gate nodes whose parents are the
    previous-step hidden node of the layer and the input from below (the layer
    below at the same step, or the step's input node), then a cell-state node
    (parents: the gates and the previous cell state) and a hidden node
    (parents: the gates). The decoder starts from the encoder's last states.
    One attention node per decoder step has all top-layer encoder hidden nodes
    and that step's top decoder hidden node as parents (fan-in steps+1); it is
    a leaf (no input feeding), which keeps the depth near two levels per
    unrolled step. `seed` is unused: the structure is deterministic; it is
    accepted for a uniform signature.
    """
    del seed
    b = _Builder()

    def lstm_cell(below: int, h_prev, c_prev):
        gate_parents = [below] + ([h_prev] if h_prev is not None else [])
        gates = [b.node(*gate_parents) for _ in range(4)]
        c = b.node(*gates, *([c_prev] if c_prev is not None else []))
        h = b.node(*gates)
        return h, c

    enc_h = [[None] * enc_layers for _ in range(steps)]
    enc_c = [[None] * enc_layers for _ in range(steps)]
    for t in range(steps):
        below = b.node()                       # source token embedding
        for l in range(enc_layers):
            hp = enc_h[t - 1][l] if t > 0 else None
            cp = enc_c[t - 1][l] if t > 0 else None
            h, c = lstm_cell(below, hp, cp)
            enc_h[t][l], enc_c[t][l] = h, c
            below = h
    enc_top = [enc_h[t][enc_layers - 1] for t in range(steps)]

    dec_h = [[None] * dec_layers for _ in range(steps)]
    dec_c = [[None] * dec_layers for _ in range(steps)]
    for t in range(steps):
        below = b.node()                       # target token embedding
        for l in range(dec_layers):
            le = min(l, enc_layers - 1)
            hp = dec_h[t - 1][l] if t > 0 else enc_h[steps - 1][le]
            cp = dec_c[t - 1][l] if t > 0 else enc_c[steps - 1][le]
            h, c = lstm_cell(below, hp, cp)
            dec_h[t][l], dec_c[t][l] = h, c
            below = h
        b.node(*enc_top, dec_h[t][dec_layers - 1])
    return b.done()


_NAS_OPS = (1, 3, 16, 16, 16, 4)   # identity, pool, sep-conv 3/5/7, 1x1 conv
_NAS_OPS_SHORT = (1, 2, 8, 8, 8, 3)


def nasnet_shaped(seed: int = 4, cells: int = 18, blocks: int = 5, ops=_NAS_OPS, adapter: int = 4,
                  lanes: int = 1):
    """A stack of NAS cells.

    A cell adapts the outputs of the two preceding cells through 1x1 adapter
    chains (`adapter` nodes each). Each of its blocks picks two inputs uniformly
    among the adapted inputs and the outputs of earlier blocks of the cell, passes
    each through an op drawn uniformly from {identity: 1 node, pool, separable
    conv with kernel 3/5/7, 1x1 conv} (chain lengths in `ops`) and adds them.
    Block outputs nobody used are joined by the cell's concat node. With
    `lanes` > 1 every op but the identity runs as that many parallel chains
    (a grouped execution of the op) that meet in the block's add node.

    The default (chains of 3 / 16 / 4, one lane) reaches the ~2000 nodes of the
    configuration by lengthening the chains: depth 744. `nasnet_shaped_wide`
    keeps chains of 2 / 8 / 3 and reaches the same size with two lanes per op:
    half the depth, twice the level width.
    """
    rng = _rng(seed)
    b = _Builder()
    prev2 = b.node()
    prev1 = b.node(prev2)
    for _ in range(cells):
        hidden = [b.chain(prev1, adapter), b.chain(prev2, adapter)]
        used = [False, False]
        for _ in range(blocks):
            ends = []
            for _ in range(2):
                pick = int(rng.integers(0, len(hidden)))
                used[pick] = True
                op = ops[int(rng.integers(0, len(ops)))]
                for _ in range(1 if op == 1 else lanes):
                    ends.append(b.chain(hidden[pick], op))
            hidden.append(b.node(*ends))
            used.append(False)
        loose = [h for h, u in zip(hidden[2:], used[2:]) if not u]
        out = b.node(*loose)
        prev2, prev1 = prev1, out
    return b.done()


def nasnet_shaped_wide(seed: int = 4):
    """The NAS-cell stack with the shorter op chains (pool 2, separable conv 8,
    1x1 conv 3, adapters 3) and two lanes per op: about the same node count as
    `nasnet_shaped`, half its depth."""
    return nasnet_shaped(seed, ops=_NAS_OPS_SHORT, adapter=3, lanes=2)


def enas_conv_shaped(seed: int, target_n: int):
    """ENAS-style convolutional network: a stack of random cells.

    Node j of a cell picks one or two predecessors among the earlier nodes of
    the cell and the outputs of the two previous cells; nodes without a
    consumer are joined by the cell's concat node. Cells are appended until
    `target_n` nodes are reached.
    """
    rng = _rng(seed)
    b = _Builder()
    prev2 = b.node()
    prev1 = b.node(prev2)
    while b.n < target_n:
        size = int(rng.integers(6, 13))
        pool = [prev1, prev2]
        used = [True, True]
        for _ in range(size):
            k = int(rng.integers(1, 3))
            picks = rng.choice(len(pool), size=min(k, len(pool)), replace=False)
            v = b.node(*[pool[int(p)] for p in picks])
            for p in picks:
                used[int(p)] = True
            pool.append(v)
            used.append(False)
        loose = [p for p, u in zip(pool, used) if not u]
        out = b.node(*loose)
        prev2, prev1 = prev1, out
    return b.done()


def enas_rnn_shaped(seed: int, target_n: int):
    """ENAS-style recurrent network: one random cell unrolled L steps.

    The cell has an input node x[t] and a first node fed by x[t] and the
    previous step's output; every further node picks one earlier node of the
    cell (its op kind, one of four, does not change the structure); nodes
    without a consumer are averaged by the step's output node. L is uniform in
    {25..40} as for the paper's ptb family (Appendix A.3); the cell size
    follows from `target_n`.
    """
    rng = _rng(seed)
    b = _Builder()
    L = int(rng.integers(25, 41))
    size = max(2, int(round(target_n / L)) - 2)
    picks = [int(rng.integers(0, j + 1)) for j in range(size - 1)]
    _kinds = rng.integers(0, 4, size=size)       # drawn to keep the recipe's draw order
    h_prev = None
    for _ in range(L):
        x = b.node()
        first = b.node(x, *([h_prev] if h_prev is not None else []))
        nodes = [first]
        used = [False]
        for j in range(size - 1):
            nodes.append(b.node(nodes[picks[j]]))
            used[picks[j]] = True
            used.append(False)
        loose = [v for v, u in zip(nodes, used) if not u]
        h_prev = b.node(*loose)
    return b.done()


def sweep_graph(i: int, count: int = 64, n_lo: int = 100, n_hi: int = 1000):
    """Graph i of the full-episode sweep: target sizes log-spaced n_lo..n_hi,
    conv-style for even i, recurrent for odd i, seed 1000+i."""
    target = int(round(n_lo * (n_hi / n_lo) ** (i / max(count - 1, 1))))
    if i % 2 == 0:
        return enas_conv_shaped(1000 + i, target)
    return enas_rnn_shaped(1000 + i, target)


def topological_order(n: int, src, dst) -> np.ndarray:
    """A topological order of the DAG (Kahn's algorithm, FIFO from ascending
    ids); raises ValueError on a cycle."""
    indeg = np.zeros(n, dtype=np.int64)
    out: list[list[int]] = [[] for _ in range(n)]
    for u, v in set(zip(map(int, src), map(int, dst))):
        out[u].append(v)
        indeg[v] += 1
    queue = [v for v in range(n) if indeg[v] == 0]
    order = []
    head = 0
    while head < len(queue):
        u = queue[head]
        head += 1
        order.append(u)
        for v in sorted(out[u]):
            indeg[v] -= 1
            if indeg[v] == 0:
                queue.append(v)
    if len(order) != n:
        raise ValueError("graph has a cycle")
    return np.asarray(order, dtype=np.int32)


def depth(n: int, src, dst) -> int:
    """Number of levels of the longest-path layering."""
    order = topological_order(n, src, dst)
    par: list[list[int]] = [[] for _ in range(n)]
    for u, v in zip(map(int, src), map(int, dst)):
        par[v].append(u)
    lvl = np.zeros(n, dtype=np.int64)
    for v in order:
        if par[v]:
            lvl[v] = 1 + max(lvl[u] for u in par[v])
    return int(lvl.max()) + 1 if n else 0
