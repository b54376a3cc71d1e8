"""ctypes front end of the CPU checker (test infrastructure only).

Compiles ``placeto_oracle.c`` with gcc on first use (double precision, and a
single-precision copy used as a rounding canary) and exposes numpy-in /
numpy-out functions. Nothing here is used by the CUDA library; only tests, the
smoke check and the benchmark's CPU-baseline leg import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "placeto_oracle.c")
_LIBS: dict[str, ctypes.CDLL] = {}


class _Mlp(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("in_dim", ctypes.c_int32),
                ("hidden_dim", ctypes.c_int32), ("out_dim", ctypes.c_int32),
                ("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p),
                ("W2", ctypes.c_void_p), ("b2", ctypes.c_void_p),
                ("act", ctypes.c_int32), ("final_act", ctypes.c_int32)]


def build(force: bool = False) -> None:
    """Compiles both precisions next to the source (no-op when up to date)."""
    for real in ("double", "float"):
        out = os.path.join(_HERE, "libplaceto_oracle_%s.so" % real)
        if (not force and os.path.exists(out)
                and os.path.getmtime(out) >= os.path.getmtime(_SRC)):
            continue
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-DORACLE_REAL=%s" % real, _SRC, "-o", out + ".tmp%d" % os.getpid(), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(out + ".tmp%d" % os.getpid(), out)


def _lib(real: str) -> ctypes.CDLL:
    if real not in _LIBS:
        build()
        lib = ctypes.CDLL(os.path.join(_HERE, "libplaceto_oracle_%s.so" % real))
        for fn in ("oracle_features", "oracle_embed", "oracle_embed_sync",
                   "oracle_policy", "oracle_group_sizes", "oracle_real_bytes"):
            getattr(lib, fn).restype = ctypes.c_int
        _LIBS[real] = lib
    return _LIBS[real]


def _dtype(real: str):
    return np.float64 if real == "double" else np.float32


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _mlp(net: dict, keep: list) -> _Mlp:
    """Packs one network dict (see gen.states.mlp_weights) into the C struct."""
    arrs = {}
    for k in ("W1", "b1", "W2", "b2"):
        a = net.get(k)
        if a is not None:
            a = np.ascontiguousarray(a, dtype=np.float32)
            keep.append(a)
        arrs[k] = a
    return _Mlp(net["n_layers"], net["in_dim"], net["hidden_dim"], net["out_dim"],
                _ptr(arrs["W1"]), _ptr(arrs["b1"]), _ptr(arrs["W2"]), _ptr(arrs["b2"]),
                net["act"], net["final_act"])


def _edges(src, dst):
    s = np.ascontiguousarray(src, dtype=np.int32)
    t = np.ascontiguousarray(dst, dtype=np.int32)
    return s, t, ctypes.c_int64(len(s))


def _check(rc: int) -> None:
    if rc != 0:
        raise ValueError({-1: "edge id out of range or self-loop", -2: "graph has a cycle",
                          -3: "current node out of range"}.get(rc, "oracle error %d" % rc))


def features(n, m, cost, nbytes, dev, cur, placed, real="double"):
    """Raw feature tensor X[n][B][m+4] (Sec. 2.2 step 1)."""
    B = dev.shape[0]
    X = np.empty((n, B, m + 4), dtype=_dtype(real))
    _check(_lib(real).oracle_features(
        ctypes.c_int32(n), ctypes.c_int32(B), ctypes.c_int32(m),
        _ptr(np.ascontiguousarray(cost, np.float32)), _ptr(np.ascontiguousarray(nbytes, np.float32)),
        _ptr(np.ascontiguousarray(dev, np.uint8)), _ptr(np.ascontiguousarray(cur, np.int32)),
        _ptr(np.ascontiguousarray(placed, np.uint8)), _ptr(X)))
    return X


def embed(n, src, dst, X, weights, real="double", threads=1):
    """Two-way message passing (Sec. 2.2 step 2): returns H_down, H_up [n][B][d]."""
    X = np.ascontiguousarray(X, dtype=_dtype(real))
    _, B, F = X.shape
    d = weights["d"]
    keep: list = []
    nets = [_mlp(weights[k], keep) for k in ("f_down", "g_down", "f_up", "g_up")]
    Hd = np.zeros((n, B, d), dtype=_dtype(real))
    Hu = np.zeros((n, B, d), dtype=_dtype(real))
    s, t, ne = _edges(src, dst)
    _check(_lib(real).oracle_embed(
        ctypes.c_int32(n), ne, _ptr(s), _ptr(t), ctypes.c_int32(B), ctypes.c_int32(F),
        ctypes.c_int32(d), _ptr(X), *[ctypes.byref(x) for x in nets], _ptr(Hd), _ptr(Hu),
        ctypes.c_int32(threads)))
    return Hd, Hu


def embed_sync(n, src, dst, X, weights, rounds, real="double"):
    """The synchronous k-round form of the message passing, from zeros."""
    X = np.ascontiguousarray(X, dtype=_dtype(real))
    _, B, F = X.shape
    d = weights["d"]
    keep: list = []
    nets = [_mlp(weights[k], keep) for k in ("f_down", "g_down", "f_up", "g_up")]
    Hd = np.zeros((n, B, d), dtype=_dtype(real))
    Hu = np.zeros((n, B, d), dtype=_dtype(real))
    s, t, ne = _edges(src, dst)
    _check(_lib(real).oracle_embed_sync(
        ctypes.c_int32(n), ne, _ptr(s), _ptr(t), ctypes.c_int32(B), ctypes.c_int32(F),
        ctypes.c_int32(d), _ptr(X), *[ctypes.byref(x) for x in nets],
        ctypes.c_int32(rounds), _ptr(Hd), _ptr(Hu)))
    return Hd, Hu


def policy(n, src, dst, X, Hd, Hu, cur, weights, real="double", threads=1):
    """Group pooling + head + softmax (Sec. 2.2 step 3, Appendix A.7):
    returns logits, probs [B][m]."""
    dt = _dtype(real)
    X = np.ascontiguousarray(X, dtype=dt)
    Hd = np.ascontiguousarray(Hd, dtype=dt)
    Hu = np.ascontiguousarray(Hu, dtype=dt)
    _, B, F = X.shape
    d, m = weights["d"], weights["m"]
    keep: list = []
    l = (_Mlp * 3)(*[_mlp(w, keep) for w in weights["l"]])
    h = (_Mlp * 3)(*[_mlp(w, keep) for w in weights["h"]])
    head = _mlp(weights["head"], keep)
    logits = np.zeros((B, m), dtype=dt)
    probs = np.zeros((B, m), dtype=dt)
    s, t, ne = _edges(src, dst)
    cur = np.ascontiguousarray(cur, dtype=np.int32)
    _check(_lib(real).oracle_policy(
        ctypes.c_int32(n), ne, _ptr(s), _ptr(t), ctypes.c_int32(B), ctypes.c_int32(F),
        ctypes.c_int32(d), ctypes.c_int32(m), _ptr(X), _ptr(Hd), _ptr(Hu), _ptr(cur),
        l, h, ctypes.byref(head), _ptr(logits), _ptr(probs), ctypes.c_int32(threads)))
    return logits, probs


def groups(n, src, dst, c):
    """Group of every node relative to c: 0 can reach c, 1 reachable from c,
    2 neither, 3 c itself; plus the three set sizes."""
    s, t, ne = _edges(src, dst)
    sizes = np.zeros(3, dtype=np.int32)
    group = np.zeros(n, dtype=np.uint8)
    _check(_lib("double").oracle_group_sizes(
        ctypes.c_int32(n), ne, _ptr(s), _ptr(t), ctypes.c_int32(int(c)), _ptr(sizes), _ptr(group)))
    return group, sizes


def forward(cfg: dict, real="double", threads=1, states=None):
    """Whole path on a configuration dict from gen.configs: features, both
    passes, pooling, head. `states` selects a subset of the batch (states are
    independent). Returns a dict of X, H_down, H_up, logits, probs."""
    dev, cur, placed = cfg["dev"], cfg["cur"], cfg["placed"]
    if states is not None:
        idx = np.asarray(states)
        dev, cur, placed = dev[idx], cur[idx], placed[idx]
    X = features(cfg["n"], cfg["m"], cfg["cost"], cfg["bytes"], dev, cur, placed, real)
    Hd, Hu = embed(cfg["n"], cfg["src"], cfg["dst"], X, cfg["weights"], real, threads)
    logits, probs = policy(cfg["n"], cfg["src"], cfg["dst"], X, Hd, Hu, cur,
                           cfg["weights"], real, threads)
    return {"X": X, "H_down": Hd, "H_up": Hu, "logits": logits, "probs": probs}
