"""REINFORCE on the device, end to end, with the library's entry points:

    sampled episodes (placeto_episode_rollout)
      -> simulated run times of the final placements (placeto_simulate_runtime)
      -> advantages = -(run time) minus the batch mean (terminal reward, Appendix A.3)
      -> policy gradient over every visited state (placeto_policy_gradient)
      -> an Adam ascent step on the weights (torch.optim: the optimiser is the caller's).

Only the glue between the calls is PyTorch: rebuilding the E * n visited states
from the actions, the advantage arithmetic and the optimiser. Run as

    python -m paper_1906_08879_b200.examples.reinforce_demo [iterations]
"""
from __future__ import annotations

import sys

import numpy as np
import torch

import paper_1906_08879_b200 as placeto


def visited_states(order, dev0, actions):
    """The E * n states an episode batch went through, as (dev, cur, placed) with
    state index e * n + t: the first t nodes of the order carry their chosen
    device and the visited flag, the rest their initial device."""
    E, n = dev0.shape
    order = order.long()
    step_of = torch.empty(n, dtype=torch.long, device=dev0.device)
    step_of[order] = torch.arange(n, device=dev0.device)             # step at which a node is visited
    by_node = torch.empty_like(actions)
    by_node[:, order] = actions                                       # the device a node ends up on
    t = torch.arange(n, device=dev0.device).view(1, n, 1)
    done = step_of.view(1, 1, n) < t                                  # [1][t][node]
    dev = torch.where(done, by_node.view(E, 1, n), dev0.view(E, 1, n)).reshape(E * n, n).contiguous()
    placed = done.expand(E, n, n).reshape(E * n, n).to(torch.uint8).contiguous()
    cur = order.to(torch.int32).view(1, n).expand(E, n).reshape(E * n).contiguous()
    return dev, cur, placed


def train(cfg, iterations=40, episodes=64, bandwidth=1.0, lr=0.002, beta=0.01, seed=0, log=None):
    """Runs REINFORCE on cfg's graph; returns the mean simulated run time per iteration."""
    n, m = cfg["n"], cfg["m"]
    dev_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    grads = placeto.binding.zero_gradients(cfg["weights"])
    names = sorted(w.tensors, key=str)
    params = [w.tensors[k] for k in names]
    opt = torch.optim.Adam(params, lr=lr)
    cost, nbytes = dev_t(cfg["cost"]), dev_t(cfg["bytes"])
    order = dev_t(np.asarray(cfg["order"], dtype=np.int32))
    gen = torch.Generator(device="cuda").manual_seed(seed)
    history = []
    for it in range(iterations):
        dev0 = torch.zeros((episodes, n), dtype=torch.uint8, device="cuda")      # everything on device 0
        uniforms = torch.rand((episodes, n), generator=gen, device="cuda")
        dev = dev0.clone()
        dev, actions, _ = placeto.placeto_episode_rollout(g, w, cost, nbytes, order, dev, uniforms)
        runtime = placeto.placeto_simulate_runtime(g, cost, nbytes, dev, m, bandwidth)
        reward = -runtime.float()
        adv = (reward - reward.mean()).view(episodes, 1).expand(episodes, n).reshape(-1).contiguous()
        sdev, scur, splaced = visited_states(order, dev0, actions)
        X = placeto.placeto_build_features(g, cost, nbytes, sdev, scur, splaced, m)
        Hd, Hu = placeto.placeto_embed_forward(g, w, X)
        placeto.placeto_policy_gradient(g, w, X, Hd, Hu, scur, actions.reshape(-1).to(torch.int32).contiguous(),
                                        adv, beta, grads)
        for k, p in zip(names, params):
            p.grad = -grads.tensors[k] / episodes        # Adam minimises: ascend the objective
        opt.step()
        history.append(float(runtime.mean()))
        if log:
            log("iteration %3d  mean simulated run time %.4f  best %.4f" % (it, history[-1], float(runtime.min())))
    return history


def demo_config(seed=0, n=14, m=2, d=32):
    """A small random DAG whose transfers are expensive next to its operations."""
    from gen import graphs, states
    r = np.random.Generator(np.random.PCG64(seed))
    src, dst = [], []
    for v in range(1, n):
        for u in r.choice(v, size=min(v, int(r.integers(1, 3))), replace=False):
            src.append(int(u)); dst.append(v)
    src, dst = np.asarray(src, np.int32), np.asarray(dst, np.int32)
    cfg = {"n": n, "src": src, "dst": dst, "m": m, "d": d, "F": m + 4}
    cfg["cost"] = r.uniform(0.5, 1.5, n).astype(np.float32)
    cfg["bytes"] = r.uniform(0.5, 1.5, n).astype(np.float32)
    cfg["weights"] = states.policy_weights(r, d, m + 4, m, 2, 0, 0.1)
    cfg["order"] = graphs.topological_order(n, src, dst)
    return cfg


if __name__ == "__main__":
    its = int(sys.argv[1]) if len(sys.argv) > 1 else 40
    lr = float(sys.argv[2]) if len(sys.argv) > 2 else 0.002
    beta = float(sys.argv[3]) if len(sys.argv) > 3 else 0.01
    train(demo_config(), iterations=its, lr=lr, beta=beta, log=print)
