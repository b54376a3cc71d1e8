"""Pins of the CPU checker against what the paper and the mathematics fix.

Each test ties oracle/placeto_oracle.c to something other than itself: exact
brute-force recursion, closed forms for linear networks, a hand-worked
fixture, invariants stated in the paper, textbook special cases.
"""
from __future__ import annotations

import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from gen import configs, graphs, states
from oracle import brute, oracle
from tests.helpers import closure, int_weights, net, random_dag, rng, row_rel_err

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- helpers ---

def _collapse(nt):
    """Affine map (W, b) of a network whose activation is the identity."""
    W, b = nt["W1"].astype(np.float64), nt["b1"].astype(np.float64)
    if nt["n_layers"] == 2:
        b = b @ nt["W2"].astype(np.float64) + nt["b2"].astype(np.float64)
        W = W @ nt["W2"].astype(np.float64)
    return W, b


def _linear_weights(r, d, F, m, layers, nonneg=False, act=1):
    w = states.policy_weights(r, d, F, m, layers, act, 0.1)
    if nonneg:
        for k, v in w.items():
            nets = v if isinstance(v, list) else [v]
            for nt in nets:
                if isinstance(nt, dict):
                    for key in ("W1", "b1", "W2", "b2"):
                        if nt.get(key) is not None:
                            nt[key] = np.abs(nt[key])
    return w


def _solve_linear(n, src, dst, X, f, g, down=True):
    """Closed form for affine f, g on any DAG:
    H = P^T H A + P^T X C + deg (x) (bf Wg) + 1 (x) bg  (row-major vec)."""
    d = g["out_dim"]
    Wf, bf = _collapse(f)
    Wg, bg = _collapse(g)
    A, C = Wf[:d] @ Wg, Wf[d:] @ Wg
    P = np.zeros((n, n))
    for u, v in set(zip(map(int, src), map(int, dst))):
        if down:
            P[u, v] = 1.0
        else:
            P[v, u] = 1.0
    deg = P.sum(axis=0)
    out = np.empty((n, X.shape[1], d))
    M = np.eye(n * d) - np.kron(P.T, A.T)
    for b in range(X.shape[1]):
        R = P.T @ X[:, b, :] @ C + np.outer(deg, bf @ Wg) + bg[None, :]
        out[:, b, :] = np.linalg.solve(M, R.reshape(-1)).reshape(n, d)
    return out


# ------------------------------------------------- P1: exact brute force ---

def _exact_case(n, src, dst, seed, d=2, m=2, layers=2):
    r = rng(seed)
    F = m + 4
    w = int_weights(r, d, F, m, layers)
    B = 3
    cost = r.integers(0, 4, size=n).astype(np.float32)
    nbytes = r.integers(0, 4, size=n).astype(np.float32)
    dev, cur, placed = states.random_states(r, n, m, B)
    X = oracle.features(n, m, cost, nbytes, dev, cur, placed)
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    logits, _ = oracle.policy(n, src, dst, X, Hd, Hu, cur, w)
    bw = {k: v for k, v in w.items()}
    br = brute.Brute(n, zip(src, dst), bw)
    for b in range(B):
        x = brute.features(m, cost, nbytes, dev[b], int(cur[b]), placed[b])
        for v in range(n):
            assert [Fraction(float(t)) for t in X[v, b]] == x[v]
            assert [Fraction(float(t)) for t in Hd[v, b]] == br.h(v, x, True), (n, v, b)
            assert [Fraction(float(t)) for t in Hu[v, b]] == br.h(v, x, False), (n, v, b)
        assert [Fraction(float(t)) for t in logits[b]] == br.logits(x, int(cur[b]))


def test_brute_force_all_four_node_dags():
    pairs = [(i, j) for i in range(4) for j in range(i + 1, 4)]
    perms = [(0, 1, 2, 3), (2, 0, 3, 1), (3, 2, 1, 0)]
    for mask in range(1 << len(pairs)):
        perm = perms[mask % 3]
        src = np.asarray([perm[p[0]] for k, p in enumerate(pairs) if mask >> k & 1], dtype=np.int32)
        dst = np.asarray([perm[p[1]] for k, p in enumerate(pairs) if mask >> k & 1], dtype=np.int32)
        _exact_case(4, src, dst, 100 + mask, layers=1 + mask % 2)


@pytest.mark.parametrize("n,seed", [(5, 1), (6, 2), (7, 3), (8, 4), (8, 5)])
def test_brute_force_random_small_dags(n, seed):
    r = rng(seed)
    src, dst = random_dag(r, n, 0.4)
    # a repeated edge must count once (neighbours are sets)
    if len(src):
        src, dst = np.append(src, src[0]), np.append(dst, dst[0])
    _exact_case(n, src, dst, 50 + seed, d=3, m=2)


# ------------------------------------ P2: chain closed form (linear f, g) ---

@pytest.mark.parametrize("layers", [1, 2])
def test_chain_closed_form(layers):
    n, d, m, B = 9, 4, 3, 2
    F = m + 4
    r = rng(7)
    w = _linear_weights(r, d, F, m, layers)
    src = np.arange(n - 1, dtype=np.int32)
    dst = src + 1
    X = r.normal(size=(n, B, F))
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    for name, H, order in (("down", Hd, list(range(n))), ("up", Hu, list(range(n - 1, -1, -1)))):
        Wf, bf = _collapse(w["f_" + name])
        Wg, bg = _collapse(w["g_" + name])
        A, C, c = Wf[:d] @ Wg, Wf[d:] @ Wg, bf @ Wg + bg
        for b in range(B):
            # h_0 = bg;  h_i = bg A^i + sum_{j<i} (x_j C + c) A^{i-1-j}   (row vectors)
            for i, v in enumerate(order):
                h = bg @ np.linalg.matrix_power(A, i)
                for j in range(i):
                    h = h + (X[order[j], b] @ C + c) @ np.linalg.matrix_power(A, i - 1 - j)
                np.testing.assert_allclose(H[v, b], h, rtol=1e-10, atol=1e-12)


# ---------------------------- P3 / P5: linear solve on general DAGs -------

@pytest.mark.parametrize("relu_inactive", [False, True])
def test_general_dag_linear_solve(relu_inactive):
    n, d, m, B = 12, 3, 2, 2
    F = m + 4
    r = rng(11)
    src, dst = random_dag(r, n, 0.3)
    if relu_inactive:
        # all weights, biases and features >= 0: ReLU never clips, so the ReLU
        # code path must reproduce the affine closed form
        w = _linear_weights(r, d, F, m, 2, nonneg=True, act=0)
        X = np.abs(r.normal(size=(n, B, F)))
    else:
        w = _linear_weights(r, d, F, m, 2, act=1)
        X = r.normal(size=(n, B, F))
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    np.testing.assert_allclose(Hd, _solve_linear(n, src, dst, X, w["f_down"], w["g_down"], True),
                               rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(Hu, _solve_linear(n, src, dst, X, w["f_up"], w["g_up"], False),
                               rtol=1e-9, atol=1e-10)


# ------------------------------------------ P4: path counting + fixture ---

def _path_count_weights():
    one = net([[1.0], [1.0]], [0.0], act=1)
    idn = net([[1.0]], [0.0], act=1)
    w = {"d": 1, "F": 1, "m": 2, "f_down": one, "g_down": idn, "f_up": one, "g_up": idn}
    return w


def test_diamond_fixture():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "diamond_path_count.txt"))
            if l.strip() and not l.startswith("#")]
    x = np.asarray([float(r[1]) for r in rows]).reshape(4, 1, 1)
    src = np.asarray([0, 0, 1, 2], dtype=np.int32)
    dst = np.asarray([1, 2, 3, 3], dtype=np.int32)
    Hd, Hu = oracle.embed(4, src, dst, x, _path_count_weights())
    assert Hd[:, 0, 0].tolist() == [float(r[2]) for r in rows]
    assert Hu[:, 0, 0].tolist() == [float(r[3]) for r in rows]


def test_path_counting():
    n = 10
    r = rng(5)
    src, dst = random_dag(r, n, 0.45)
    src, dst = np.append(src, src[:2]), np.append(dst, dst[:2])   # repeats count once
    x = r.integers(-3, 4, size=(n, 1, 1)).astype(np.float64)
    Hd, Hu = oracle.embed(n, src, dst, x, _path_count_weights())
    P = np.zeros((n, n))
    P[src, dst] = 1.0
    paths = np.linalg.inv(np.eye(n) - P) - np.eye(n)       # paths[u][v] = #paths u -> v
    np.testing.assert_allclose(Hd[:, 0, 0], paths.T @ x[:, 0, 0], atol=1e-9)
    np.testing.assert_allclose(Hu[:, 0, 0], paths @ x[:, 0, 0], atol=1e-9)


# -------------------------------------------- P6: relabelling invariance ---

def test_relabelling_invariance():
    cfg = configs.make("tiny")
    ref = oracle.forward(cfg)
    r = rng(3)
    n = cfg["n"]
    perm = r.permutation(n).astype(np.int32)            # old id -> new id
    shuffle = r.permutation(len(cfg["src"]))
    c2 = dict(cfg)
    c2["src"], c2["dst"] = perm[cfg["src"]][shuffle], perm[cfg["dst"]][shuffle]
    inv = np.argsort(perm)
    c2["cost"], c2["bytes"] = cfg["cost"][inv], cfg["bytes"][inv]
    c2["dev"], c2["placed"] = cfg["dev"][:, inv], cfg["placed"][:, inv]
    c2["cur"] = perm[cfg["cur"]]
    out = oracle.forward(c2)
    assert row_rel_err(out["H_down"][perm], ref["H_down"]) < 1e-12
    assert row_rel_err(out["H_up"][perm], ref["H_up"]) < 1e-12
    assert row_rel_err(out["logits"], ref["logits"]) < 1e-11
    assert row_rel_err(out["probs"], ref["probs"]) < 1e-9


# --------------------------------- P7: synchronous rounds = progressive ---

def test_synchronous_rounds_reach_progressive_sweep():
    cfg = configs.make("tiny", normalise=True)
    X = oracle.features(cfg["n"], cfg["m"], cfg["cost"], cfg["bytes"], cfg["dev"], cfg["cur"], cfg["placed"])
    args = (cfg["n"], cfg["src"], cfg["dst"], X, cfg["weights"])
    Hd, Hu = oracle.embed(*args)
    depth = cfg["depth"]
    Sd, Su = oracle.embed_sync(*args, rounds=depth)
    np.testing.assert_array_equal(Sd, Hd)
    np.testing.assert_array_equal(Su, Hu)
    Sd2, Su2 = oracle.embed_sync(*args, rounds=depth + 3)       # a fixed point
    np.testing.assert_array_equal(Sd2, Hd)
    np.testing.assert_array_equal(Su2, Hu)
    Sd3, _ = oracle.embed_sync(*args, rounds=depth - 1)         # one round short
    assert not np.array_equal(Sd3, Hd)


@pytest.mark.parametrize("layers", [1, 2])
def test_synchronous_rounds_truncated_series(layers):
    """Finite k (Sec. 2.2 step 2: the update repeated k times, from zeros). For
    affine f and g one round is H <- P^T H A + T with T = P^T X C + deg (x) c + 1 (x) b_g,
    so k rounds give the k-term series  sum_{j<k} (P^T)^j T A^j:  matrix powers,
    no iteration. Fixes the values at k = 1, 2, 3 (below the depth)."""
    n, d, m, B = 12, 3, 2, 2
    F = m + 4
    r = rng(41)
    src, dst = random_dag(r, n, 0.3)
    w = _linear_weights(r, d, F, m, layers)
    X = r.normal(size=(n, B, F))
    for k in (0, 1, 2, 3):
        Sd, Su = oracle.embed_sync(n, src, dst, X, w, rounds=k)
        for name, S, down in (("down", Sd, True), ("up", Su, False)):
            Wf, bf = _collapse(w["f_" + name])
            Wg, bg = _collapse(w["g_" + name])
            A, C = Wf[:d] @ Wg, Wf[d:] @ Wg
            P = np.zeros((n, n))
            for u, v in set(zip(map(int, src), map(int, dst))):
                P[(u, v) if down else (v, u)] = 1.0
            deg = P.sum(axis=0)
            for b in range(B):
                T = P.T @ X[:, b, :] @ C + np.outer(deg, bf @ Wg) + bg[None, :]
                want = np.zeros((n, d))
                for j in range(k):
                    want += np.linalg.matrix_power(P.T, j) @ T @ np.linalg.matrix_power(A, j)
                np.testing.assert_allclose(S[:, b, :], want, rtol=1e-10, atol=1e-12)


# ---------------------------------------------------- P8: influence sets ---

def test_influence_sets():
    n, d, m = 14, 4, 2
    F = m + 4
    r = rng(21)
    src, dst = random_dag(r, n, 0.2)
    # identity activation and positive weights: every path carries influence
    w = _linear_weights(r, d, F, m, 1, nonneg=True, act=1)
    X = np.abs(r.normal(size=(n, 1, F))) + 0.5
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    R = closure(n, src, dst)
    for u in range(n):
        X2 = X.copy()
        X2[u] += 1.0
        Hd2, Hu2 = oracle.embed(n, src, dst, X2, w)
        changed_d = np.any(Hd2 != Hd, axis=(1, 2))
        changed_u = np.any(Hu2 != Hu, axis=(1, 2))
        np.testing.assert_array_equal(changed_d, R[u, :])     # strict descendants of u hear it top-down
        np.testing.assert_array_equal(changed_u, R[:, u])     # strict ancestors hear it bottom-up


# ------------------------------------------------ P9: partition identity ---

def test_groups_partition_and_match_closure():
    cfg = configs.make("inception")
    n = cfg["n"]
    R = closure(n, cfg["src"], cfg["dst"])
    for c in (0, 17, 100, n - 1):
        group, sizes = oracle.groups(n, cfg["src"], cfg["dst"], c)
        assert sizes.sum() == n - 1 and group[c] == 3
        np.testing.assert_array_equal(group == 0, R[:, c])
        np.testing.assert_array_equal(group == 1, R[c, :])


def test_pooling_sum_identity():
    """Equal l for the three groups and identity h: the three pooled vectors
    plus l(e_c) add up to the sum of l(e_u) over all nodes."""
    n, d, m, B = 11, 3, 2, 4
    F = m + 4
    r = rng(31)
    src, dst = random_dag(r, n, 0.25)
    w = states.policy_weights(r, d, F, m, 2, 0, 0.1)
    w["l"] = [w["l"][0]] * 3
    eye = net(np.eye(d), np.zeros(d), act=1)
    w["h"] = [eye] * 3
    Z = 5 * d + F
    # head reads the three pooled vectors through an identity-like first layer
    W1 = np.zeros((Z, Z)); W1[np.arange(Z), np.arange(Z)] = 1.0
    W2 = np.zeros((Z, d))
    for i in range(3):
        W2[2 * d + F + i * d + np.arange(d), np.arange(d)] = 1.0
    w["head"] = net(W1, np.zeros(Z), W2, np.zeros(d), act=1, final_act=0)
    w["m"] = d
    X = r.normal(size=(n, B, F))
    cur = r.integers(0, n, size=B).astype(np.int32)
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    logits, _ = oracle.policy(n, src, dst, X, Hd, Hu, cur, w)
    E = np.concatenate([Hd, Hu, X], axis=2)
    L = np.maximum(E @ w["l"][0]["W1"].astype(np.float64) + w["l"][0]["b1"], 0.0)   # [n][B][d]
    for b in range(B):
        total = L[:, b].sum(axis=0) - L[cur[b], b]
        np.testing.assert_allclose(logits[b], total, rtol=1e-10, atol=1e-10)


# --------------------------------------- P10: textbook special cases -------

def test_single_node_is_plain_mlp():
    d, m, B = 5, 3, 3
    F = m + 4
    r = rng(41)
    w = states.policy_weights(r, d, F, m, 2, 0, 0.1)
    X = r.normal(size=(1, B, F))
    e = np.zeros(0, dtype=np.int32)
    Hd, Hu = oracle.embed(1, e, e, X, w)
    cur = np.zeros(B, dtype=np.int32)
    logits, probs = oracle.policy(1, e, e, X, Hd, Hu, cur, w)
    relu = lambda t: np.maximum(t, 0.0)
    g0 = lambda g: relu(relu(g["b1"].astype(np.float64)) @ g["W2"] + g["b2"])
    for b in range(B):
        np.testing.assert_allclose(Hd[0, b], g0(w["g_down"]), rtol=1e-12)
        np.testing.assert_allclose(Hu[0, b], g0(w["g_up"]), rtol=1e-12)
        z = np.concatenate([Hd[0, b], Hu[0, b], X[0, b]]
                           + [relu(w["h"][i]["b1"].astype(np.float64)) for i in range(3)])
        hd = w["head"]
        lg = relu(z @ hd["W1"] + hd["b1"]) @ hd["W2"] + hd["b2"]
        np.testing.assert_allclose(logits[b], lg, rtol=1e-12)
        p = np.exp(lg - lg.max()); p /= p.sum()
        np.testing.assert_allclose(probs[b], p, rtol=1e-12)


def test_roots_and_leaves_share_the_bias_only_embedding():
    cfg = configs.make("tiny", normalise=True)
    out = oracle.forward(cfg)
    n = cfg["n"]
    roots = sorted(set(range(n)) - set(cfg["dst"].tolist()))
    leaves = sorted(set(range(n)) - set(cfg["src"].tolist()))
    assert len(roots) >= 2 and len(leaves) >= 2
    for v in roots:
        np.testing.assert_array_equal(out["H_down"][v], out["H_down"][roots[0]])
    for v in leaves:
        np.testing.assert_array_equal(out["H_up"][v], out["H_up"][leaves[0]])
    assert np.ptp(out["H_down"][roots[0]], axis=0).max() == 0      # same for every state


def test_softmax_properties():
    cfg = configs.make("tiny", normalise=True)
    out = oracle.forward(cfg)
    np.testing.assert_allclose(out["probs"].sum(axis=1), 1.0, rtol=1e-12)
    assert (out["probs"].argmax(axis=1) == out["logits"].argmax(axis=1)).all()
    # shifting the head's output bias by a constant leaves the probabilities alone
    c2 = dict(cfg); w2 = dict(cfg["weights"]); hd = dict(w2["head"])
    hd["b2"] = hd["b2"] + np.float32(3.0)
    w2["head"] = hd; c2["weights"] = w2
    out2 = oracle.forward(c2)
    np.testing.assert_allclose(out2["probs"], out["probs"], rtol=1e-6)
    np.testing.assert_allclose(out2["logits"], out["logits"] + 3.0, rtol=1e-6)


def test_simple_partitioner_special_case():
    """With the embedding columns of l_i and of the head zeroed, the policy is
    the paper's 'simple partitioner' ablation (Sec. 4.2): per-group pooling of
    raw features only, computed here directly with numpy."""
    n, d, m, B = 13, 4, 3, 5
    F = m + 4
    r = rng(51)
    src, dst = random_dag(r, n, 0.25)
    w = states.policy_weights(r, d, F, m, 2, 0, 0.1)
    for nt in w["l"]:
        nt["W1"][: 2 * d] = 0
    w["head"]["W1"][: 2 * d] = 0
    cost, nbytes = states.node_costs(r, n, normalise=True)
    dev, cur, placed = states.random_states(r, n, m, B)
    X = oracle.features(n, m, cost, nbytes, dev, cur, placed)
    Hd, Hu = oracle.embed(n, src, dst, X, w)
    logits, _ = oracle.policy(n, src, dst, X, Hd, Hu, cur, w)
    R = closure(n, src, dst)
    relu = lambda t: np.maximum(t, 0.0)
    for b in range(B):
        c = int(cur[b])
        sets = [R[:, c], R[c, :], ~(R[:, c] | R[c, :])]
        sets[2][c] = False
        z = [np.zeros(2 * d), X[c, b]]
        for i in range(3):
            s = sum((relu(X[u, b] @ w["l"][i]["W1"][2 * d:].astype(np.float64) + w["l"][i]["b1"])
                     for u in np.nonzero(sets[i])[0]), np.zeros(d))
            z.append(relu(s @ w["h"][i]["W1"].astype(np.float64) + w["h"][i]["b1"]))
        z = np.concatenate(z)
        hd = w["head"]
        lg = relu(z @ hd["W1"].astype(np.float64) + hd["b1"]) @ hd["W2"].astype(np.float64) + hd["b2"]
        np.testing.assert_allclose(logits[b], lg, rtol=1e-10, atol=1e-12)


# ------------------------------------------------ features + P11 + misc ---

def test_feature_layout():
    n, m, B = 6, 3, 4
    r = rng(61)
    cost, nbytes = states.node_costs(r, n)
    dev, cur, placed = states.random_states(r, n, m, B)
    X = oracle.features(n, m, cost, nbytes, dev, cur, placed)
    assert X.shape == (n, B, m + 4)
    for v, b in itertools.product(range(n), range(B)):
        x = X[v, b]
        assert x[0] == np.float64(cost[v]) and x[1] == np.float64(nbytes[v])
        assert x[2:2 + m].sum() == 1 and x[2 + dev[b, v]] == 1
        assert x[2 + m] == (cur[b] == v) and x[3 + m] == placed[b, v]


def test_batch_independence():
    cfg = configs.make("tiny")
    full = oracle.forward(cfg)
    for sel in ([5], [9, 2, 2]):
        part = oracle.forward(cfg, states=sel)
        np.testing.assert_array_equal(part["H_down"], full["H_down"][:, sel])
        np.testing.assert_array_equal(part["H_up"], full["H_up"][:, sel])
        np.testing.assert_array_equal(part["logits"], full["logits"][sel])


def test_rejects_cycle_and_bad_ids():
    X = np.zeros((3, 1, 1))
    w = _path_count_weights()
    with pytest.raises(ValueError):
        oracle.embed(3, np.asarray([0, 1, 2], np.int32), np.asarray([1, 2, 0], np.int32), X, w)
    with pytest.raises(ValueError):
        oracle.embed(3, np.asarray([0], np.int32), np.asarray([3], np.int32), X, w)
    with pytest.raises(ValueError):
        oracle.embed(3, np.asarray([1], np.int32), np.asarray([1], np.int32), X, w)


def test_threads_do_not_change_results():
    cfg = configs.make("tiny")
    a = oracle.forward(cfg, threads=1)
    b = oracle.forward(cfg, threads=4)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_single_precision_canary_close_to_double():
    cfg = configs.make("tiny", normalise=True)
    a = oracle.forward(cfg)
    b = oracle.forward(cfg, real="float")
    assert row_rel_err(b["H_down"], a["H_down"]) < 1e-4
    assert row_rel_err(b["logits"], a["logits"]) < 1e-4


def test_episode_states_follow_the_mdp():
    """Sec. 2.1: one node is current per step, visited nodes are the ones
    before it in the traversal, |V| steps."""
    n, src, dst = graphs.sweep_graph(0)
    r = rng(1)
    dev, cur, placed = states.episode_states(r, n, src, dst, 8)
    assert sorted(cur.tolist()) == list(range(n))
    pos = np.argsort(cur)
    for u, v in zip(src, dst):
        assert pos[u] < pos[v]
    for t in range(n):
        assert placed[t].sum() == t and placed[t, cur[t]] == 0
        assert (dev[t][placed[t] == 0] == 0).all()
