"""GPU parity of placeto_simple_aggregator (the "simple aggregator" ablation of
Sec. 4.3) against oracle/aggregator.py on the same seeded inputs; tolerances as
in tests/test_gpu_parity.py."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs
from oracle import aggregator, oracle
from tests.helpers import net, rng, row_rel_err

pytestmark = pytest.mark.gpu


def _weights(r, F, d, m, hidden, l_layers=1, head_layers=2):
    def W(a, b):
        lim = np.sqrt(6.0 / (a + b))
        return r.uniform(-lim, lim, size=(a, b)).astype(np.float32)

    def bias(a):
        return r.uniform(-0.1, 0.1, size=a).astype(np.float32)

    l = net(W(F, d), bias(d)) if l_layers == 1 else net(W(F, F), bias(F), W(F, d), bias(d))
    head = (net(W(d, hidden), bias(hidden), W(hidden, m), bias(m), final_act=0) if head_layers == 2
            else net(W(d, m), bias(m), final_act=0))
    return {"d": d, "F": F, "m": m, "l": l, "h": net(W(d, d), bias(d)), "head": head}


def _check(cfg, w):
    X64 = oracle.features(cfg["n"], cfg["m"], cfg["cost"], cfg["bytes"], cfg["dev"], cfg["cur"], cfg["placed"])
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    X = torch.from_numpy(X64.astype(np.float32)).cuda()
    logits, probs = placeto.placeto_simple_aggregator(g, placeto.AggregatorWeights(w), X)
    torch.cuda.synchronize()
    ref_logits, ref_probs = aggregator.simple_aggregator(X64, w)
    got = logits.cpu().numpy()
    assert np.isfinite(got).all()
    assert row_rel_err(got, ref_logits, 0.1) <= 1e-4 and row_rel_err(got, ref_logits, 1.0) <= 2e-5
    np.testing.assert_allclose(probs.cpu().numpy().sum(axis=1), 1.0, rtol=1e-5)
    calm = np.abs(ref_logits).max(axis=1) < 50.0
    if calm.any():
        np.testing.assert_allclose(probs.cpu().numpy()[calm], ref_probs[calm], atol=5e-4)
    # twice the same bits
    logits2, _ = placeto.placeto_simple_aggregator(g, placeto.AggregatorWeights(w), X)
    assert torch.equal(logits, logits2)


@pytest.mark.parametrize("name,d,hidden,l_layers,head_layers", [
    ("tiny", 8, 6, 1, 2), ("tiny", 8, 6, 2, 1), ("inception", 32, 32, 1, 2), ("inception", 128, 1024, 2, 2),
    ("nmt", 20, 17, 1, 2)])
def test_simple_aggregator_matches_the_checker(name, d, hidden, l_layers, head_layers):
    cfg = configs.make(name, normalise=True)
    w = _weights(rng(d + hidden), cfg["F"], d, cfg["m"], hidden, l_layers, head_layers)
    _check(cfg, w)


def test_simple_aggregator_on_raw_feature_scale_and_argument_errors():
    cfg = configs.make("tiny")
    w = _weights(rng(3), cfg["F"], 8, cfg["m"], 8)
    _check(cfg, w)
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    bad = dict(w, d=9)                        # networks no longer fit d
    X = torch.zeros((cfg["n"], 4, cfg["F"]), device="cuda")
    with pytest.raises(placeto.PlacetoError) as e:
        placeto.placeto_simple_aggregator(g, placeto.AggregatorWeights(bad), X)
    assert e.value.status == 1
