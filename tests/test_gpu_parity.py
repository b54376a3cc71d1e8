"""GPU parity: the CUDA library, called through its C ABI, against the CPU
checker on the same seeded inputs, element by element.

Tolerances (fp32 path): for every output row (the d-vector of one node and
state, or the m logits of one state)
    max_i |gpu_i - ref_i| / max(|ref_i|, 0.1 * ||ref row||_inf)  <= 1e-4
and, normwise,
    max_i |gpu_i - ref_i| / ||ref row||_inf                      <= 2e-5.
The device argmax must equal the checker's wherever the checker's top-2 logit
gap exceeds max(1e-3, 2e-5 * ||logits||_inf) (the second term is the normwise
tolerance: below it fp32 cannot resolve the order at the raw feature scale).
"""
from __future__ import annotations

import ctypes

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs, states
from oracle import oracle
from tests.helpers import net, random_dag, rng, row_rel_err

pytestmark = pytest.mark.gpu

TOL_ELEM, TOL_NORM = 1e-4, 2e-5
SCHEDULES = {"sliced": placeto.PLACETO_SLICED, "per_level": placeto.PLACETO_PER_LEVEL,
             "cooperative": placeto.PLACETO_COOPERATIVE,
             "generic_sliced": placeto.PLACETO_SLICED | placeto.PLACETO_GENERIC,
             "fma_only": placeto.PLACETO_FMA_ONLY, "tensor": placeto.PLACETO_TENSOR,
             "tcgen05": placeto.PLACETO_TCGEN05, "pipeline": placeto.PLACETO_PIPELINE}


def dev_t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_close(got, ref, what):
    got = got.detach().cpu().numpy() if isinstance(got, torch.Tensor) else got
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what
    e1 = row_rel_err(got, ref, 0.1)
    e2 = row_rel_err(got, ref, 1.0)
    assert e1 <= TOL_ELEM and e2 <= TOL_NORM, "%s: elementwise %.3g normwise %.3g" % (what, e1, e2)


def assert_argmax(logits, ref_logits):
    logits = logits.detach().cpu().numpy()
    srt = np.sort(ref_logits, axis=1)
    gap = srt[:, -1] - srt[:, -2] if ref_logits.shape[1] > 1 else np.full(len(srt), np.inf)
    need = gap > np.maximum(1e-3, TOL_NORM * np.abs(ref_logits).max(axis=1))
    same = logits.argmax(axis=1) == ref_logits.argmax(axis=1)
    assert same[need].all(), "argmax differs on %d decisive states" % int((~same[need]).sum())
    return int(need.sum())


def gpu_forward(cfg, flags=0, sel=None):
    """features -> embed -> logits through the three C entry points."""
    devs, cur, placed = cfg["dev"], cfg["cur"], cfg["placed"]
    if sel is not None:
        devs, cur, placed = devs[sel], cur[sel], placed[sel]
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    cur_d = dev_t(cur)
    X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(devs),
                                       cur_d, dev_t(placed), cfg["m"])
    Hd, Hu = placeto.placeto_embed_forward(g, w, X, flags=flags)
    logits, probs = placeto.placeto_policy_logits(g, w, X, Hd, Hu, cur_d, flags=flags)
    torch.cuda.synchronize()
    return {"X": X, "H_down": Hd, "H_up": Hu, "logits": logits, "probs": probs, "graph": g, "w": w}


def compare(cfg, out, ref, sel=None):
    pick = (lambda t: t) if sel is None else (lambda t: t[:, sel])
    np.testing.assert_array_equal(pick(out["X"]).cpu().numpy(), ref["X"].astype(np.float32))
    assert_close(pick(out["H_down"]), ref["H_down"], "H_down")
    assert_close(pick(out["H_up"]), ref["H_up"], "H_up")
    lg = out["logits"] if sel is None else out["logits"][sel]
    pr = out["probs"] if sel is None else out["probs"][sel]
    assert_close(lg, ref["logits"], "logits")
    assert_argmax(lg, ref["logits"])
    p = pr.cpu().numpy()
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-5)
    # probabilities follow the logits: compare against the softmax of the device logits
    l64 = lg.cpu().numpy().astype(np.float64)
    sm = np.exp(l64 - l64.max(axis=1, keepdims=True))
    sm /= sm.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(p, sm, atol=2e-6)
    # and the checker's where the logit error cannot move them
    scale = np.abs(ref["logits"]).max(axis=1)
    calm = scale < 50.0
    if calm.any():
        np.testing.assert_allclose(p[calm], ref["probs"][calm], atol=5e-4)


# ------------------------------------------------------------ the configs ---

@pytest.mark.parametrize("schedule", list(SCHEDULES))
@pytest.mark.parametrize("normalise", [False, True])
def test_tiny(schedule, normalise):
    cfg = configs.make("tiny", normalise=normalise)
    out = gpu_forward(cfg, SCHEDULES[schedule])
    compare(cfg, out, oracle.forward(cfg))


@pytest.mark.parametrize("schedule", list(SCHEDULES))
def test_inception(schedule):
    cfg = configs.make("inception")
    out = gpu_forward(cfg, SCHEDULES[schedule])
    compare(cfg, out, oracle.forward(cfg, threads=8))


def test_inception_normalised():
    cfg = configs.make("inception", normalise=True)
    compare(cfg, gpu_forward(cfg), oracle.forward(cfg, threads=8))


@pytest.mark.parametrize("flags", [0, placeto.PLACETO_TENSOR])
@pytest.mark.parametrize("normalise", [False, True])
def test_nmt(normalise, flags):
    cfg = configs.make("nmt", normalise=normalise)
    out = gpu_forward(cfg, flags)
    compare(cfg, out, oracle.forward(cfg, threads=8))


@pytest.mark.parametrize("flags", [0, placeto.PLACETO_FMA_ONLY, placeto.PLACETO_TENSOR, placeto.PLACETO_TCGEN05])
def test_nasnet_full_batch_sampled_states(flags):
    """Full size on the GPU (n ~ 2100, B = 512, d = 64); the checker evaluates
    a sample of states one by one (states are independent). At this batch the
    tensor-core kernels give a block a slice of 8 (mma.sync) or 7 (tcgen05)
    states that share the rows of a tile: the sample holds every position of a
    slice (states 0..7 and 504..511 under either slicing) and states from the
    middle of the batch."""
    cfg = configs.make("nasnet")
    out = gpu_forward(cfg, flags)
    sel = np.asarray(list(range(8)) + [63, 64, 255, 258, 259, 261, 300, 448] + list(range(504, 512)))
    compare(cfg, out, oracle.forward(cfg, threads=8, states=sel), sel=sel)
    for k in ("H_down", "H_up", "logits", "probs"):
        assert torch.isfinite(out[k]).all()


def _sweep_case(i, flags, samples):
    cfg = configs.make_sweep(i)
    out = gpu_forward(cfg, flags)
    n = cfg["n"]
    sel = None if n <= 320 else np.unique(np.linspace(0, n - 1, samples).astype(int))
    ref = oracle.forward(cfg, threads=8, states=sel)
    compare(cfg, out, ref, sel=sel)


@pytest.mark.parametrize("i", range(64))
def test_episode_sweep(i):
    """Every graph of the full-episode sweep, all |V| states on the GPU; the
    checker takes all of them up to 320 nodes and 24 evenly spaced ones beyond."""
    _sweep_case(i, 0, 24)


@pytest.mark.parametrize("i", [0, 1, 30, 63])
def test_episode_sweep_on_the_tensor_kernel(i):
    _sweep_case(i, placeto.PLACETO_TENSOR, 48)


# ------------------------------------------------------------- edge cases ---

def _small_case(n, src, dst, d=8, m=3, B=5, layers=2, act=0, seed=0, schedule=0, F=None):
    r = rng(seed)
    F_ = m + 4
    cfg = {"n": n, "src": np.asarray(src, np.int32), "dst": np.asarray(dst, np.int32), "m": m,
           "d": d, "F": F_}
    cfg["cost"], cfg["bytes"] = states.node_costs(r, n, normalise=True)
    cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(r, n, m, B)
    cfg["weights"] = states.policy_weights(r, d, F_, m, layers, act, 0.1)
    out = gpu_forward(cfg, schedule)
    compare(cfg, out, oracle.forward(cfg))


@pytest.mark.parametrize("schedule", list(SCHEDULES))
def test_degenerate_graphs(schedule):
    s = SCHEDULES[schedule]
    e = np.zeros(0, np.int32)
    _small_case(1, e, e, schedule=s)                                   # one node
    _small_case(5, e, e, schedule=s)                                   # no edges
    _small_case(9, np.arange(8), np.arange(1, 9), schedule=s)          # chain
    _small_case(7, np.zeros(6, np.int32), np.arange(1, 7), schedule=s) # star out
    _small_case(7, np.arange(1, 7), np.zeros(6, np.int32), schedule=s) # star in (fan-in 6)
    _small_case(4, [0, 0, 1, 2, 0], [1, 2, 3, 3, 1], schedule=s)       # diamond, repeated edge
    _small_case(7, [0, 1, 3, 4], [1, 2, 4, 5], schedule=s)             # components + isolated


@pytest.mark.parametrize("B", [1, 2, 31, 33, 77, 300])
def test_ragged_batches(B):
    r = rng(B)
    src, dst = random_dag(r, 40, 0.1)
    _small_case(40, src, dst, d=16, m=4, B=B, seed=B)


@pytest.mark.parametrize("d,m", [(1, 1), (3, 2), (8, 2), (20, 5), (32, 4), (48, 8), (64, 8), (128, 6)])
def test_widths(d, m):
    r = rng(7)
    src, dst = random_dag(r, 24, 0.15)
    _small_case(24, src, dst, d=d, m=m, B=9, seed=d)


@pytest.mark.parametrize("d", [32, 64])
@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 8, 11, 12])
def test_specialised_kernels_over_feature_widths(d, m):
    """F = m + 4 from 5 to 16: vector and scalar feature prefetch, every padded
    first-layer width of the d = 32 / 64 kernels, pooling with and without the
    fast path (it needs F to be a multiple of 4)."""
    r = rng(100 * d + m)
    n = int(r.integers(30, 90))
    src, dst = random_dag(r, n, float(r.uniform(0.03, 0.12)))
    B = int(r.integers(3, 70))
    for flags in (0, placeto.PLACETO_FMA_ONLY, placeto.PLACETO_TENSOR, placeto.PLACETO_TCGEN05,
                  placeto.PLACETO_PIPELINE):
        _small_case(n, src, dst, d=d, m=m, B=B, seed=m + d, schedule=flags)


@pytest.mark.parametrize("B", [1, 7, 33, 300, 1200])
def test_tcgen05_kernel_over_batch_sizes(B):
    """d = 64 on tcgen05: one state per block, ragged last slice, slices of up to
    17 states (tiles of more than 32 and more than 64 rows on the wide levels)."""
    r = rng(B)
    src, dst = random_dag(r, 60, 0.08)
    _small_case(60, src, dst, d=64, m=8, B=B, seed=B, schedule=placeto.PLACETO_TCGEN05)


@pytest.mark.parametrize("B", [1, 7, 33, 300, 1200])
def test_pipeline_kernel_over_batch_sizes(B):
    """d = 64 as a pipeline of layers: one state per block (a tile holds rows of up to
    eight nodes), a ragged last slice, and slices of up to 17 states, forced by the flag
    (levels of more tiles than a ring holds, so tiles enter while others leave)."""
    r = rng(B)
    src, dst = random_dag(r, 60, 0.08)
    _small_case(60, src, dst, d=64, m=8, B=B, seed=B, schedule=placeto.PLACETO_PIPELINE)


@pytest.mark.parametrize("B", [3, 40])
def test_pipeline_kernel_on_degenerate_graphs(B):
    """One node, no edges (one level of several tiles), chain, stars (fan-in 6: the gather's
    neighbour loop), repeated edge, components: d = 64 through the pipeline of layers."""
    s = placeto.PLACETO_PIPELINE
    e = np.zeros(0, np.int32)
    for n, src, dst in ((1, e, e), (5, e, e), (9, np.arange(8), np.arange(1, 9)),
                        (7, np.zeros(6, np.int32), np.arange(1, 7)), (7, np.arange(1, 7), np.zeros(6, np.int32)),
                        (4, [0, 0, 1, 2, 0], [1, 2, 3, 3, 1]), (7, [0, 1, 3, 4], [1, 2, 4, 5])):
        _small_case(n, src, dst, d=64, m=4, B=B, seed=n + B, schedule=s)


def test_pipeline_kernel_on_a_deep_chain_and_a_wide_level():
    n = 1500
    src = list(range(n - 1)) + list(range(0, n - 40, 37))
    dst = list(range(1, n)) + [i + 40 for i in range(0, n - 40, 37)]
    _small_case(n, src, dst, d=64, m=8, B=10, seed=29, schedule=placeto.PLACETO_PIPELINE)
    # 40 roots -> 12 nodes -> 1 sink with 20 states per block: levels of 100 and 30 tiles
    r = rng(31)
    src = list(range(40)) + [40 + i for i in range(12)]
    dst = [40 + int(r.integers(0, 12)) for _ in range(40)] + [52] * 12
    _small_case(53, src, dst, d=64, m=12, B=1480, seed=31, schedule=placeto.PLACETO_PIPELINE)


def test_tcgen05_kernel_on_a_deep_chain_and_a_wide_level():
    n = 1500
    src = list(range(n - 1)) + list(range(0, n - 40, 37))
    dst = list(range(1, n)) + [i + 40 for i in range(0, n - 40, 37)]
    _small_case(n, src, dst, d=64, m=8, B=10, seed=29, schedule=placeto.PLACETO_TCGEN05)
    # 40 roots -> 12 nodes -> 1 sink with 20 states per block: levels of 800 and 240 rows
    r = rng(31)
    src = list(range(40)) + [40 + i for i in range(12)]
    dst = [40 + int(r.integers(0, 12)) for _ in range(40)] + [52] * 12
    _small_case(53, src, dst, d=64, m=12, B=1480, seed=31, schedule=placeto.PLACETO_TCGEN05)


def test_error_channel_reports_a_wait_that_ran_out():
    """A kernel whose barrier can never complete gives up after a bounded number of
    polls and reports it; the record is tied to its call, so the next call (and
    a workspace full of whatever memory held before) reads as clean. Nothing
    faults: the same context carries on."""
    cfg = configs.make("tiny")
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    ws = placeto.workspace(g, w, cfg["B"], placeto.CALL_FORWARD)
    ws.fill_(0xAB)
    assert placeto.placeto_last_status(g, ws) == 0
    placeto.placeto_debug_wait_timeout(g, ws)
    assert placeto.placeto_last_status(g, ws) == 8
    assert placeto.binding.status_string(8) == "a bounded wait inside a kernel ran out"
    out = gpu_forward(cfg)
    compare(cfg, out, oracle.forward(cfg))
    logits, _ = placeto.placeto_policy_forward(g, w, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]),
                                               dev_t(cfg["cur"]), dev_t(cfg["placed"]), ws=ws)
    assert placeto.placeto_last_status(g, ws) == 0
    assert torch.equal(logits, out["logits"])


@pytest.mark.parametrize("name", ["tiny", "inception", "nmt", "nasnet", "sweep63"])
def test_error_at_the_one_percent_floor_beside_the_single_precision_checker(name, capsys):
    """The gates above put the floor of the elementwise error at 0.1 of the row's
    largest entry. With the floor at 0.01 the error of ANY fp32 evaluation grows
    (small entries of a row carry the row's absolute error): the library's figure
    is reported beside that of the checker compiled in single precision and held
    to three times it."""
    cfg = configs.make_sweep(63) if name == "sweep63" else configs.make(name)
    B = cfg["B"]
    sel = None if B <= 16 else np.unique(np.linspace(0, B - 1, 16).astype(int))
    out = gpu_forward(cfg)
    ref = oracle.forward(cfg, threads=8, states=sel)
    can = oracle.forward(cfg, real="float", threads=8, states=sel)
    worst = 0.0
    lines = []
    for key in ("H_down", "H_up", "logits"):
        got = out[key].cpu().numpy()
        if sel is not None:
            got = got[:, sel] if key != "logits" else got[sel]
        e_gpu = row_rel_err(got, ref[key], 0.01)
        e_can = row_rel_err(can[key], ref[key], 0.01)
        lines.append("%s %s: library %.3g, single-precision checker %.3g" % (name, key, e_gpu, e_can))
        worst = max(worst, e_gpu / max(3.0 * e_can, 1e-5))
    with capsys.disabled():
        print("\n[0.01 floor] " + "; ".join(lines))
    assert worst <= 1.0, lines


def test_single_layer_networks_as_in_the_paper():
    """Appendix A.7: single-layer f, g (hidden = input width)."""
    r = rng(9)
    src, dst = random_dag(r, 30, 0.12)
    for sched in SCHEDULES.values():
        _small_case(30, src, dst, d=16, m=4, B=12, layers=1, seed=3, schedule=sched)


def test_identity_activation_and_path_counting():
    one = net([[1.0], [1.0]], [0.0], act=1)
    idn = net([[1.0]], [0.0], act=1)
    w = {"d": 1, "F": 1, "m": 2, "f_down": one, "g_down": idn, "f_up": one, "g_up": idn}
    src = np.asarray([0, 0, 1, 2], np.int32)
    dst = np.asarray([1, 2, 3, 3], np.int32)
    x = np.asarray([3.0, 5.0, -4.0, 11.0], np.float32).reshape(4, 1, 1)
    g = placeto.Graph(4, src, dst)
    Hd, Hu = placeto.placeto_embed_forward(g, placeto.Weights(w), dev_t(x))
    assert Hd.cpu().numpy()[:, 0, 0].tolist() == [0.0, 3.0, 3.0, 7.0]
    assert Hu.cpu().numpy()[:, 0, 0].tolist() == [23.0, 11.0, 11.0, 0.0]


def test_max_fan_in_node():
    n = 130
    src = np.arange(n - 1)
    dst = np.full(n - 1, n - 1)
    _small_case(n, src, dst, d=32, m=4, B=20, seed=5)


@pytest.mark.parametrize("d,m", [(32, 4), (64, 8)])
def test_very_wide_level_falls_back_to_the_generic_kernel(d, m):
    """2000 roots -> 40 nodes -> 1 sink: the message slots of one level exceed
    shared memory, so the specialised kernels decline and the generic one runs."""
    r = rng(17)
    roots, mid = 2000, 40
    src = list(range(roots)) + [roots + i for i in range(mid)]
    dst = [roots + int(r.integers(0, mid)) for _ in range(roots)] + [roots + mid] * mid
    _small_case(roots + mid + 1, src, dst, d=d, m=m, B=24, seed=23)


@pytest.mark.parametrize("d,m", [(32, 4), (64, 8)])
def test_long_chain_with_skips(d, m):
    """Depth 1500: many levels of one node, plus skip edges that keep messages alive."""
    n = 1500
    src = list(range(n - 1)) + list(range(0, n - 40, 37))
    dst = list(range(1, n)) + [i + 40 for i in range(0, n - 40, 37)]
    _small_case(n, src, dst, d=d, m=m, B=10, seed=29)


# ------------------------------------------------------ properties on GPU ---

def test_deterministic_and_batch_independent():
    cfg = configs.make("inception")
    a = gpu_forward(cfg)
    b = gpu_forward(cfg)
    for k in ("H_down", "H_up", "logits", "probs"):
        assert torch.equal(a[k], b[k]), k
    sel = np.asarray([200, 3, 77])
    c = gpu_forward(cfg, sel=sel)
    for k in ("H_down", "H_up"):
        assert_close(c[k], a[k][:, sel].cpu().numpy().astype(np.float64), k)
    assert_close(c["logits"], a["logits"][sel].cpu().numpy().astype(np.float64), "logits")


def test_relabelling_invariance_on_gpu():
    cfg = configs.make("inception", normalise=True)
    ref = gpu_forward(cfg)
    r = rng(3)
    n = cfg["n"]
    perm = r.permutation(n).astype(np.int32)
    inv = np.argsort(perm)
    c2 = dict(cfg)
    sh = r.permutation(len(cfg["src"]))
    c2["src"], c2["dst"] = perm[cfg["src"]][sh], perm[cfg["dst"]][sh]
    c2["cost"], c2["bytes"] = cfg["cost"][inv], cfg["bytes"][inv]
    c2["dev"], c2["placed"] = cfg["dev"][:, inv], cfg["placed"][:, inv]
    c2["cur"] = perm[cfg["cur"]]
    out = gpu_forward(c2)
    perm_t = torch.from_numpy(perm.astype(np.int64)).cuda()
    assert_close(out["H_down"][perm_t], ref["H_down"].cpu().numpy().astype(np.float64), "H_down")
    assert_close(out["logits"], ref["logits"].cpu().numpy().astype(np.float64), "logits")


def test_schedules_agree():
    cfg = configs.make("nmt", B=24)
    outs = [gpu_forward(cfg, s) for s in SCHEDULES.values()]
    ref = oracle.forward(cfg, threads=8)
    for o in outs:
        compare(cfg, o, ref)


# ------------------------------------------------- synchronous k rounds ---

@pytest.mark.parametrize("d,m,layers", [(8, 3, 2), (32, 4, 2), (32, 4, 1), (64, 8, 2)])
def test_synchronous_rounds_against_the_checker(d, m, layers):
    """placeto_embed_rounds: H^0 = 0, every node updated at once from the
    previous round, k rounds (the form Sec. 2.2 step 2 states)."""
    r = rng(31 * d + layers)
    n, B = 22, 13
    src, dst = random_dag(r, n, 0.15)
    F = m + 4
    cost, nbytes = states.node_costs(r, n, normalise=True)
    devs, cur, placed = states.random_states(r, n, m, B)
    weights = states.policy_weights(r, d, F, m, layers, 0, 0.1)
    g = placeto.Graph(n, src, dst)
    w = placeto.Weights(weights)
    X = placeto.placeto_build_features(g, dev_t(cost), dev_t(nbytes), dev_t(devs), dev_t(cur),
                                       dev_t(placed), m)
    Xh = X.cpu().numpy().astype(np.float64)
    depth = g.info()["n_levels_down"]
    for k in (0, 1, 2, 3, depth, depth + 2):
        Hd, Hu = placeto.placeto_embed_rounds(g, w, X, k)
        torch.cuda.synchronize()
        assert placeto.placeto_last_launch_count() == (k + 1 if k else 0)
        rd, ru = oracle.embed_sync(n, src, dst, Xh, weights, k)
        assert_close(Hd, rd, "H_down after %d rounds" % k)
        assert_close(Hu, ru, "H_up after %d rounds" % k)
    # from depth rounds on the synchronous form has reached the progressive sweep
    Pd, Pu = placeto.placeto_embed_forward(g, w, X)
    torch.cuda.synchronize()
    assert_close(Hd, Pd.cpu().numpy().astype(np.float64), "rounds vs sweep, down")
    assert_close(Hu, Pu.cpu().numpy().astype(np.float64), "rounds vs sweep, up")


def test_synchronous_rounds_on_the_inception_shaped_graph():
    cfg = configs.make("inception", B=40, normalise=True)
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]),
                                       dev_t(cfg["cur"]), dev_t(cfg["placed"]), cfg["m"])
    Hd, Hu = placeto.placeto_embed_rounds(g, w, X, 3)
    torch.cuda.synchronize()
    rd, ru = oracle.embed_sync(cfg["n"], cfg["src"], cfg["dst"], X.cpu().numpy().astype(np.float64),
                               cfg["weights"], 3)
    assert_close(Hd, rd, "H_down")
    assert_close(Hu, ru, "H_up")


def test_simple_partitioner_variant_is_the_pooling_on_zero_embeddings():
    """The paper's "simple partitioner" ablation (Sec. 4, alternative policy
    architectures) pools the raw features of the three sets without the message
    passing: placeto_policy_logits on zero embeddings."""
    cfg = configs.make("inception", B=24, normalise=True)
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    cur = dev_t(cfg["cur"])
    X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]),
                                       cur, dev_t(cfg["placed"]), cfg["m"])
    Z = torch.zeros((cfg["n"], 24, cfg["d"]), dtype=torch.float32, device="cuda")
    logits, probs = placeto.placeto_policy_logits(g, w, X, Z, Z, cur)
    torch.cuda.synchronize()
    zeros = np.zeros((cfg["n"], 24, cfg["d"]))
    rl, rp = oracle.policy(cfg["n"], cfg["src"], cfg["dst"], X.cpu().numpy().astype(np.float64), zeros,
                           zeros, cfg["cur"], cfg["weights"])
    assert_close(logits, rl, "logits")
    assert_argmax(logits, rl)


# ------------------------------------------------ fused and host variants ---

def test_policy_forward_and_host_variant_match_the_separate_calls():
    cfg = configs.make("inception")
    ref = gpu_forward(cfg)
    g, w = ref["graph"], ref["w"]
    B = cfg["B"]
    logits, probs = placeto.placeto_policy_forward(
        g, w, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]), dev_t(cfg["cur"]),
        dev_t(cfg["placed"]))
    torch.cuda.synchronize()
    assert torch.equal(logits, ref["logits"]) and torch.equal(probs, ref["probs"])
    assert placeto.placeto_last_launch_count() >= 4
    ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD_HOST)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_logits = torch.empty((B, cfg["m"]), dtype=torch.float32).pin_memory()
    h_probs = torch.empty((B, cfg["m"]), dtype=torch.float32).pin_memory()
    placeto.placeto_policy_forward_host(g, w, pin(cfg["cost"]), pin(cfg["bytes"]), pin(cfg["dev"]),
                                        pin(cfg["cur"]), pin(cfg["placed"]), h_logits, h_probs, ws)
    assert torch.equal(h_logits, ref["logits"].cpu()) and torch.equal(h_probs, ref["probs"].cpu())


@pytest.mark.parametrize("pinned_in,pinned_out", [(False, False), (True, False), (False, True)])
def test_host_variant_with_pageable_buffers(pinned_in, pinned_out):
    """Page-locked buffers are read and written by the kernels themselves,
    pageable ones go through copies: every mix gives the same results, also with an
    unaligned pageable input and without the probabilities."""
    cfg = configs.make("tiny")
    ref = gpu_forward(cfg)
    g, w = ref["graph"], ref["w"]
    B, m = cfg["B"], cfg["m"]
    ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD_HOST)

    def host(a, pinned, shift=0):
        a = np.ascontiguousarray(a)
        if pinned:
            return torch.from_numpy(a).pin_memory()
        raw = np.empty(a.nbytes + 64, dtype=np.uint8)      # pageable, optionally off 16-byte alignment
        off = (-raw.ctypes.data) % 16 + shift
        view = raw[off:off + a.nbytes].view(a.dtype).reshape(a.shape)
        view[...] = a
        return torch.from_numpy(view)

    ins = [host(cfg["cost"], pinned_in), host(cfg["bytes"], pinned_in), host(cfg["dev"], pinned_in, 1),
           host(cfg["cur"], pinned_in), host(cfg["placed"], pinned_in)]
    out = lambda: host(np.zeros((B, m), np.float32), pinned_out)
    h_logits, h_probs = out(), out()
    placeto.placeto_policy_forward_host(g, w, *ins, h_logits, h_probs, ws)
    assert torch.equal(h_logits, ref["logits"].cpu()) and torch.equal(h_probs, ref["probs"].cpu())
    only_logits = out()
    placeto.placeto_policy_forward_host(g, w, *ins, only_logits, None, ws)
    assert torch.equal(only_logits, ref["logits"].cpu())


def test_two_streams_with_their_own_workspaces_do_not_interfere():
    cfg = configs.make("inception")
    ref = gpu_forward(cfg)
    g, w = ref["graph"], ref["w"]
    B, m = cfg["B"], cfg["m"]
    ins = [dev_t(cfg[k]) for k in ("cost", "bytes", "dev", "cur", "placed")]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    torch.cuda.synchronize()
    for st in streams:
        ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD)
        logits = torch.empty((B, m), device="cuda")
        probs = torch.empty((B, m), device="cuda")
        for _ in range(3):
            placeto.placeto_policy_forward(g, w, *ins, logits, probs, ws, 0, st)
        outs.append((logits, probs, ws))
    torch.cuda.synchronize()
    for logits, probs, _ in outs:
        assert torch.equal(logits, ref["logits"]) and torch.equal(probs, ref["probs"])


def test_back_to_back_calls_with_inputs_changed_on_the_stream():
    """The kernels of one forward call overlap their set-up with the kernel
    before them. Nothing may be read early that an earlier kernel on the stream
    still writes: states and weights are rewritten by ordinary stream work between
    calls that share one workspace, and every call must see exactly its own."""
    cfg = configs.make("inception")
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    B, m, n = cfg["B"], cfg["m"], cfg["n"]
    r = rng(11)
    variants = [states.random_states(r, n, m, B) for _ in range(3)]
    cost, nbytes = dev_t(cfg["cost"]), dev_t(cfg["bytes"])
    originals = [t.clone() for t in w._keep]

    def set_weights(scale):
        for t, o in zip(w._keep, originals):
            t.copy_(o * scale)

    # one call at a time, synchronised: the expected results
    want = []
    for k, (devs, cur, placed) in enumerate(variants):
        set_weights(1.0 + 0.25 * k)
        torch.cuda.synchronize()
        lg, pr = placeto.placeto_policy_forward(g, w, cost, nbytes, dev_t(devs), dev_t(cur), dev_t(placed))
        torch.cuda.synchronize()
        want.append((lg.clone(), pr.clone()))
    # the same calls queued back to back on one stream with one workspace and one set of buffers
    ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD)
    d_dev = torch.empty((B, n), dtype=torch.uint8, device="cuda")
    d_cur = torch.empty((B,), dtype=torch.int32, device="cuda")
    d_placed = torch.empty((B, n), dtype=torch.uint8, device="cuda")
    staged = [(dev_t(a), dev_t(b), dev_t(c)) for a, b, c in variants]
    got = []
    torch.cuda.synchronize()
    for k, (a, b, c) in enumerate(staged):
        set_weights(1.0 + 0.25 * k)
        d_dev.copy_(a); d_cur.copy_(b); d_placed.copy_(c)
        lg = torch.empty((B, m), device="cuda")
        pr = torch.empty((B, m), device="cuda")
        placeto.placeto_policy_forward(g, w, cost, nbytes, d_dev, d_cur, d_placed, lg, pr, ws)
        got.append((lg, pr))
    torch.cuda.synchronize()
    for (lg, pr), (wl, wp) in zip(got, want):
        assert torch.equal(lg, wl) and torch.equal(pr, wp)


@pytest.mark.parametrize("B", [593, 1185])
def test_head_kernel_with_four_and_eight_states_per_block(B):
    """Batches beyond two blocks per SM at two states per block move the head
    kernel to four, then eight states per block."""
    r = rng(B)
    src, dst = random_dag(r, 20, 0.2)
    _small_case(20, src, dst, d=32, m=4, B=B, seed=B)


# ---------------------------------------------------------- error handling ---

def test_argument_errors_are_reported_not_faulted():
    cfg = configs.make("tiny")
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    B = cfg["B"]
    X = torch.zeros((cfg["n"], B, cfg["F"]), device="cuda")
    ws = placeto.workspace(g, w, B, placeto.CALL_EMBED)

    def status(fn):
        with pytest.raises(placeto.PlacetoError) as e:
            fn()
        return e.value.status
    assert status(lambda: placeto.placeto_embed_forward(g, w, X, ws=ws[: ws.numel() // 2])) == 3
    assert status(lambda: placeto.placeto_embed_forward(g, w, X, ws=ws, flags=3)) == 1
    assert status(lambda: placeto.placeto_embed_forward(g, w, X, ws=ws, flags=1 << 9)) == 1
    Xb = torch.zeros(cfg["n"] * B * cfg["F"] + 1, device="cuda")[1:].view(cfg["n"], B, cfg["F"])
    assert status(lambda: placeto.placeto_embed_forward(g, w, Xb, ws=ws)) == 1   # misaligned
    bad = dict(cfg["weights"]); bad["d"] = cfg["d"] + 1
    assert status(lambda: placeto.placeto_embed_forward(g, placeto.Weights(bad), X, ws=ws)) == 1
    # an out-of-range current node poisons that state only
    cur = cfg["cur"].copy(); cur[3] = cfg["n"] + 5
    Xf = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]),
                                        dev_t(cfg["cur"]), dev_t(cfg["placed"]), cfg["m"])
    Hd, Hu = placeto.placeto_embed_forward(g, w, Xf)
    logits, _ = placeto.placeto_policy_logits(g, w, Xf, Hd, Hu, dev_t(cur))
    good, _ = placeto.placeto_policy_logits(g, w, Xf, Hd, Hu, dev_t(cfg["cur"]))
    torch.cuda.synchronize()
    assert torch.isnan(logits[3]).all()
    keep = [i for i in range(B) if i != 3]
    assert torch.equal(logits[keep], good[keep])
