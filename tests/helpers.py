"""Shared test helpers: small weight builders, error metric, random DAGs."""
from __future__ import annotations

import numpy as np


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def net(W1, b1, W2=None, b2=None, act=0, final_act=1):
    W1 = np.asarray(W1, dtype=np.float32)
    n_layers = 1 if W2 is None else 2
    out = W1.shape[1] if W2 is None else np.asarray(W2).shape[1]
    return {"n_layers": n_layers, "in_dim": W1.shape[0], "hidden_dim": W1.shape[1],
            "out_dim": out, "W1": W1, "b1": np.asarray(b1, dtype=np.float32),
            "W2": None if W2 is None else np.asarray(W2, dtype=np.float32),
            "b2": None if b2 is None else np.asarray(b2, dtype=np.float32),
            "act": act, "final_act": final_act}


def random_dag(r, n, p=0.35):
    """Random DAG on n nodes: a random permutation gives the order, each
    forward pair is an edge with probability p. Returns (src, dst)."""
    perm = r.permutation(n)
    src, dst = [], []
    for i in range(n):
        for j in range(i + 1, n):
            if r.random() < p:
                src.append(perm[i])
                dst.append(perm[j])
    return np.asarray(src, dtype=np.int32), np.asarray(dst, dtype=np.int32)


def int_weights(r, d, F, m, mp_layers=2, act=0, lo=-2, hi=3):
    """Small-integer weights for exact arithmetic."""
    def W(a, b):
        return r.integers(lo, hi, size=(a, b)).astype(np.float32)

    def bias(a):
        return r.integers(lo, hi, size=a).astype(np.float32)

    def mk(i, h, o, layers, final_act=1):
        if layers == 1:
            return net(W(i, o), bias(o), act=act, final_act=final_act)
        return net(W(i, h), bias(h), W(h, o), bias(o), act=act, final_act=final_act)

    w = {"d": d, "F": F, "m": m}
    for name in ("down", "up"):
        w["f_" + name] = mk(d + F, d, d, mp_layers)
        w["g_" + name] = mk(d, d, d, mp_layers)
    w["l"] = [mk(2 * d + F, 0, d, 1) for _ in range(3)]
    w["h"] = [mk(d, 0, d, 1) for _ in range(3)]
    w["head"] = mk(5 * d + F, 5 * d + F, m, 2, final_act=0)
    return w


def row_rel_err(got, ref, floor=0.01):
    """max_i |got_i - ref_i| / max(|ref_i|, floor * ||row||_inf), rows taken
    along the last axis (the embedding or device vector an element belongs to)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    row = np.max(np.abs(ref), axis=-1, keepdims=True)
    den = np.maximum(np.abs(ref), floor * row)
    den = np.where(den == 0, 1.0, den)
    return float(np.max(np.abs(got - ref) / den)) if ref.size else 0.0


def closure(n, src, dst):
    """reach[u][v] = True if a path of length >= 1 leads from u to v
    (boolean matrix powers: independent of any graph traversal code)."""
    A = np.zeros((n, n), dtype=bool)
    A[np.asarray(src, dtype=int), np.asarray(dst, dtype=int)] = True
    R = A.copy()
    while True:                       # paths of length <= 2^k after k squarings
        Rf = R.astype(np.float32)
        R2 = R | ((Rf @ Rf) > 0)
        if (R2 == R).all():
            return R
        R = R2
