"""Pins of the simple-aggregator checker (oracle/aggregator.py) against what the
definition fixes: exact rational brute force, the affine closed form, the fact
that it ignores graph structure and node order, softmax properties; and two
planted mistakes that these pins catch."""
from __future__ import annotations

from fractions import Fraction

import numpy as np
import pytest

from oracle import aggregator, brute
from tests.helpers import net, rng


def _weights(r, F, d, m, hidden, act=0, integer=False):
    def W(a, b):
        return (r.integers(-2, 3, size=(a, b)) if integer else r.normal(size=(a, b)) / np.sqrt(a)).astype(np.float32)

    def bias(a):
        return (r.integers(-2, 3, size=a) if integer else r.uniform(-0.1, 0.1, size=a)).astype(np.float32)

    return {"l": net(W(F, d), bias(d), act=act), "h": net(W(d, d), bias(d), act=act),
            "head": net(W(d, hidden), bias(hidden), W(hidden, m), bias(m), act=act, final_act=0)}


def test_exact_brute_force():
    """Sum over all nodes of l(x_u), then h, then the head, in exact rationals."""
    r = rng(5)
    n, B, F, d, m = 5, 3, 4, 3, 2
    w = _weights(r, F, d, m, 4, integer=True)
    X = r.integers(-3, 4, size=(n, B, F)).astype(np.float64)
    logits, probs = aggregator.simple_aggregator(X, w)
    for b in range(B):
        s = [Fraction(0)] * d
        for u in range(n):
            y = brute.mlp(w["l"], [Fraction(int(t)) for t in X[u, b]])
            s = [p + q for p, q in zip(s, y)]
        want = brute.mlp(w["head"], brute.mlp(w["h"], s))
        assert [Fraction(float(t)) for t in logits[b]] == want
    np.testing.assert_allclose(probs.sum(axis=1), 1.0, rtol=1e-12)


def test_affine_closed_form():
    """Identity activations: logits = ((sum_u x_u) Wl + n bl) Wh + bh, through the collapsed head."""
    r = rng(6)
    n, B, F, d, m = 9, 2, 5, 4, 3
    w = _weights(r, F, d, m, 6, act=1)
    X = r.normal(size=(n, B, F))
    logits, _ = aggregator.simple_aggregator(X, w)
    f64 = lambda k, key: np.asarray(w[k][key], dtype=np.float64)
    a = (X.sum(axis=0) @ f64("l", "W1") + n * f64("l", "b1")) @ f64("h", "W1") + f64("h", "b1")
    want = (a @ f64("head", "W1") + f64("head", "b1")) @ f64("head", "W2") + f64("head", "b2")
    np.testing.assert_allclose(logits, want, rtol=1e-11, atol=1e-12)


def test_node_order_does_not_matter_and_softmax_is_a_softmax():
    r = rng(7)
    n, B, F, d, m = 12, 4, 6, 5, 4
    w = _weights(r, F, d, m, 8)
    X = r.normal(size=(n, B, F))
    logits, probs = aggregator.simple_aggregator(X, w)
    logits2, _ = aggregator.simple_aggregator(X[r.permutation(n)], w)
    np.testing.assert_allclose(logits2, logits, rtol=1e-11, atol=1e-12)
    assert (probs.argmax(axis=1) == logits.argmax(axis=1)).all()
    np.testing.assert_allclose(np.log(probs[:, 0] / probs[:, 1]), logits[:, 0] - logits[:, 1], rtol=1e-9)


@pytest.mark.parametrize("mistake", ["mean instead of sum", "l skipped"])
def test_planted_mistakes_are_caught(mistake, monkeypatch):
    if mistake == "mean instead of sum":
        def wrong(X, weights):
            X = np.asarray(X, dtype=np.float64)
            lg = np.asarray([aggregator._mlp(weights["head"], aggregator._mlp(weights["h"], np.mean(
                [aggregator._mlp(weights["l"], X[u, b]) for u in range(X.shape[0])], axis=0))) for b in range(X.shape[1])])
            e = np.exp(lg - lg.max(axis=1, keepdims=True))
            return lg, e / e.sum(axis=1, keepdims=True)
    else:
        def wrong(X, weights):
            X = np.asarray(X, dtype=np.float64)
            Wl = np.asarray(weights["l"]["W1"], dtype=np.float64)
            lg = np.asarray([aggregator._mlp(weights["head"], aggregator._mlp(weights["h"], X[:, b].sum(axis=0) @ Wl))
                             for b in range(X.shape[1])])
            e = np.exp(lg - lg.max(axis=1, keepdims=True))
            return lg, e / e.sum(axis=1, keepdims=True)
    monkeypatch.setattr(aggregator, "simple_aggregator", wrong)
    caught = 0
    for pin in (test_exact_brute_force, test_affine_closed_form):
        try:
            pin()
        except AssertionError:
            caught += 1
    assert caught >= 1
