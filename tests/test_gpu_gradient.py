"""GPU parity of placeto_policy_gradient against the CPU checker (PyTorch fp64
reverse-mode differentiation of the restated forward, pinned to the C checker).
Every gradient array must agree normwise: max |gpu - ref| <= TOL * max |ref| of
that array (fp32 sums over up to n * B rows; the forward's own normwise
tolerance is 2e-5 per row)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs, states
from oracle import gradient
from tests.helpers import random_dag, rng

pytestmark = pytest.mark.gpu

TOL = 2e-4


def dev_t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_gradient(cfg, actions, adv, beta):
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    cur = dev_t(cfg["cur"])
    X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]),
                                       cur, dev_t(cfg["placed"]), cfg["m"])
    Hd, Hu = placeto.placeto_embed_forward(g, w, X)
    grads = placeto.binding.zero_gradients(cfg["weights"])
    placeto.placeto_policy_gradient(g, w, X, Hd, Hu, cur, dev_t(actions.astype(np.int32)),
                                    dev_t(adv.astype(np.float32)), beta, grads)
    torch.cuda.synchronize()
    return grads


def compare(cfg, grads, ref):
    worst = 0.0
    for (name, idx, key), t in grads.tensors.items():
        want = ref[name][key] if idx is None else ref[name][idx][key]
        got = t.cpu().numpy().astype(np.float64)
        assert got.shape == want.shape and np.isfinite(got).all(), (name, idx, key)
        scale = np.abs(want).max()
        err = np.abs(got - want).max()
        assert err <= TOL * max(scale, 1e-6), "%s[%s].%s: error %.3g against scale %.3g" % (name, idx, key, err, scale)
        worst = max(worst, err / max(scale, 1e-30))
    return worst


def small_case(seed, n, m, d, B, p=0.2):
    r = rng(seed)
    src, dst = random_dag(r, n, p)
    cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
    cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(r, n, m, B)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.2)
    return cfg, r.integers(0, m, B), r.normal(size=B)


@pytest.mark.parametrize("d,m,B,beta", [(4, 3, 5, 0.0), (8, 2, 33, 0.5), (32, 4, 20, 0.1), (64, 8, 9, 0.0)])
def test_small_graphs(d, m, B, beta):
    cfg, actions, adv = small_case(10 * d + m, n=18, m=m, d=d, B=B)
    adv32 = adv.astype(np.float32).astype(np.float64)
    grads = gpu_gradient(cfg, actions, adv32, beta)
    compare(cfg, grads, gradient.gradient(cfg, actions, adv32, beta))


def test_degenerate_graphs_and_entropy_only():
    e = np.zeros(0, np.int32)
    for n, src, dst in ((1, e, e), (4, e, e), (6, np.arange(5, dtype=np.int32), np.arange(1, 6, dtype=np.int32))):
        r = rng(n)
        m, d, B = 3, 8, 6
        cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
        cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
        cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(r, n, m, B)
        cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.2)
        actions = r.integers(0, m, B)
        zero = np.zeros(B)
        grads = gpu_gradient(cfg, actions, zero, 1.0)
        compare(cfg, grads, gradient.gradient(cfg, actions, zero, 1.0))


def test_inception_shaped_graph():
    cfg = configs.make("inception", B=12, normalise=True)
    r = rng(4)
    actions = r.integers(0, cfg["m"], 12)
    adv = r.normal(size=12).astype(np.float32).astype(np.float64)
    grads = gpu_gradient(cfg, actions, adv, 0.05)
    compare(cfg, grads, gradient.gradient(cfg, actions, adv, 0.05))


def test_accumulating_over_two_halves_of_the_batch():
    cfg, actions, adv = small_case(12, n=16, m=4, d=32, B=24)
    adv = adv.astype(np.float32).astype(np.float64)
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    grads = placeto.binding.zero_gradients(cfg["weights"])
    for k, sel in enumerate((slice(0, 10), slice(10, 24))):
        cur = dev_t(cfg["cur"][sel])
        X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"][sel]),
                                           cur, dev_t(cfg["placed"][sel]), cfg["m"])
        Hd, Hu = placeto.placeto_embed_forward(g, w, X)
        placeto.placeto_policy_gradient(g, w, X, Hd, Hu, cur, dev_t(actions[sel].astype(np.int32)),
                                        dev_t(adv[sel].astype(np.float32)), 0.2, grads, accumulate=k > 0)
    torch.cuda.synchronize()
    compare(cfg, grads, gradient.gradient(cfg, actions, adv, 0.2))


def test_reproducible_and_unsupported_shapes():
    cfg, actions, adv = small_case(3, n=14, m=4, d=32, B=17)
    a = gpu_gradient(cfg, actions, adv, 0.1)
    b = gpu_gradient(cfg, actions, adv, 0.1)
    for key, t in a.tensors.items():
        assert torch.equal(t, b.tensors[key]), key
    # identity activations are not differentiated
    r = rng(6)
    cfg["weights"] = states.policy_weights(r, 32, 8, 4, 2, 1, 0.2)
    with pytest.raises(placeto.PlacetoError) as e:
        gpu_gradient(cfg, actions, adv, 0.0)
    assert e.value.status == 4


@pytest.mark.parametrize("d,m", [(8, 3), (32, 4)])
def test_single_layer_networks_as_in_the_paper(d, m):
    """Appendix A.7: f and g are single layers. Every gradient array against the checker."""
    cfg, actions, adv = small_case(21 + d, n=15, m=m, d=d, B=19)
    r = rng(d)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 1, 0, 0.2)
    grads = gpu_gradient(cfg, actions, adv, 0.05)
    compare(cfg, grads, gradient.gradient(cfg, actions, adv, 0.05))
