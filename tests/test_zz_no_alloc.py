"""GPU test of placeto_policy_logits_static, the entry point for callers that
cannot allocate device memory (a serving loop with a frozen memory budget, a
plug-in whose host owns the allocator). It keeps the pooling step's partial
sums in an array built into the library instead of a caller workspace, so the
array is shared by all calls and still holds the previous call's sums.

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test. The test also passes alone in a fresh
process (it does its own set-up and leans on no state of earlier tests).
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_1906_08879_b200 as placeto
from gen import configs

pytestmark = pytest.mark.gpu


def _inputs(cfg):
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    g = placeto.Graph(cfg["n"], cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    cur = t(cfg["cur"])
    X = placeto.placeto_build_features(g, t(cfg["cost"]), t(cfg["bytes"]), t(cfg["dev"]), cur,
                                       t(cfg["placed"]), cfg["m"])
    Hd, Hu = placeto.placeto_embed_forward(g, w, X)
    return g, w, X, Hd, Hu, cur


@pytest.mark.parametrize("name", ["tiny", "inception"])
def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row(name):
    cfg = configs.make(name)
    g, w, X, Hd, Hu, cur = _inputs(cfg)
    ref_logits, ref_probs = placeto.placeto_policy_logits(g, w, X, Hd, Hu, cur)
    # a second batch with other current nodes, so that the shared array holds
    # different sums between the two calls
    cur2 = torch.flip(cur, dims=[0]).contiguous()
    ref2_logits, ref2_probs = placeto.placeto_policy_logits(g, w, X, Hd, Hu, cur2)
    torch.cuda.synchronize()
    B, m = cfg["B"], cfg["m"]
    for c, want_l, want_p in ((cur, ref_logits, ref_probs), (cur2, ref2_logits, ref2_probs),
                              (cur, ref_logits, ref_probs)):
        logits = torch.full((B, m), float("nan"), device="cuda")
        probs = torch.full((B, m), float("nan"), device="cuda")
        placeto.placeto_policy_logits_static(g, w, X, Hd, Hu, c, logits, probs)
        torch.cuda.synchronize()
        # the same kernels, chunking and summation order as the workspace call: the same bits
        assert torch.equal(logits, want_l)
        assert torch.equal(probs, want_p)
        assert placeto.placeto_last_status(g, None) == 0


def test_static_scratch_call_rejects_a_batch_beyond_its_array():
    cfg = configs.make_sweep(63)                       # B = n = 992: needs more than 4 MiB
    g, w, X, Hd, Hu, cur = _inputs(cfg)
    need = placeto.placeto_workspace_bytes(g, w, cfg["B"], placeto.CALL_LOGITS)
    assert need > placeto.binding.STATIC_SCRATCH_BYTES
    logits = torch.zeros((cfg["B"], cfg["m"]), device="cuda")
    with pytest.raises(placeto.PlacetoError) as e:
        placeto.placeto_policy_logits_static(g, w, X, Hd, Hu, cur, logits)
    assert e.value.status == 7
    assert "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert (logits == 0).all()                         # nothing was launched
