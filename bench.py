#!/usr/bin/env python
"""Benchmark of the Placeto policy forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path (features -> two-way message passing ->
group pooling -> head -> softmax) over one batch of synthetic placement states
through the C ABI. The default workload is the NASNet-shaped configuration, the
largest of the five (2130 nodes in 744 levels, d = 64, 512 states); the same line
carries short measurements of the other four under "other_workloads" and the
library's error against the CPU checker on a sample of states. Prints one JSON line.

Multi-GPU (torchrun, one rank per GPU): states are independent, so every rank
runs its own batch of the same size (weak scaling) with no data-path
collective; the value is all ranks' states divided by the slowest rank's time.

`--impl reference` times the CPU checker (oracle/) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "placement-state evaluations/sec (full-graph embed + logits)"
UNIT = "evaluations/s"
FP32_LANES_PER_SM = 128           # FMA lanes per SM
L2_FLUSH_BYTES = 256 << 20        # > 126 MB L2


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="nasnet",
                    help="tiny | inception | nmt | nasnet | nasnet_wide | sweepNN")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the short measurements of the other workloads (other_workloads)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--flags", type=int, default=0, help="schedule flags of placeto.h")
    ap.add_argument("--cpu-baseline-seconds", type=float, default=10.0)
    ap.add_argument("--rounds", type=int, default=0,
                    help="K > 0: the message-passing launch timed alone (roofline) is placeto_embed_rounds "
                         "with K synchronous rounds instead of the progressive sweep")
    ap.add_argument("--gradient", action="store_true",
                    help="instead of the policy path, time placeto_policy_gradient (the backward of one batch, "
                         "embeddings given) on the workload; own JSON line")
    ap.add_argument("--simulate", type=int, default=0,
                    help="P > 0: instead of the policy path, time placeto_simulate_runtime on P random "
                         "placements of the workload's graph (its own metric: simulated placements/s)")
    ap.add_argument("--episodes", type=int, default=0,
                    help="E > 0: a step is one placeto_episode_rollout call of E sampled episodes over the "
                         "workload's graph (|V| policy evaluations per episode, transitions on the device)")
    return ap.parse_args()


def make_workload(name: str, rank: int = 0):
    from gen import configs, states
    if name.startswith("sweep"):
        cfg = configs.make_sweep(int(name[5:] or 0))
    else:
        cfg = configs.make(name)
    if rank > 0:   # other ranks: same graph and weights, their own states
        rng = np.random.Generator(np.random.PCG64(7919 * rank + 1))
        cfg["dev"], cfg["cur"], cfg["placed"] = states.random_states(rng, cfg["n"], cfg["m"], cfg["B"])
    return cfg


def workload_config(cfg, n_gpus):
    return {"workload": cfg["name"], "n_nodes": cfg["n"], "n_edges": int(len(set(zip(cfg["src"].tolist(), cfg["dst"].tolist())))),
            "depth": cfg["depth"], "d": cfg["d"], "F": cfg["F"], "m": cfg["m"],
            "states_per_gpu": cfg["B"], "global_states": cfg["B"] * n_gpus,
            "parallelism": "state batch replicated per GPU, no collective" if n_gpus > 1 else "single GPU",
            "l2": "flushed between timed steps (256 MiB memset, outside the timed events)"}


def flops_embed(cfg):
    d, F = cfg["d"], cfg["F"]
    return 2.0 * (8 * d * d + 2 * d * F) * cfg["n"] * cfg["B"]


def flops_pool(cfg):
    d, F = cfg["d"], cfg["F"]
    return 2.0 * (2 * d * d + d * F) * cfg["n"] * cfg["B"]


def job_throughput(local_ms: float, states_per_rank: int, steps: int, dist=None, device="cpu"):
    """Whole-job evaluations/s: every rank processed `states_per_rank` states per
    step; the job takes as long as its slowest rank (max over ranks of the
    device time). Returns (value, slowest_ms)."""
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    world = 1
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        world = dist.get_world_size()
    slowest = float(t.item())
    return states_per_rank * world * steps / (slowest * 1e-3), slowest


def measured_traffic(workload: str, flags: int = 0):
    """DRAM bytes per launch of the message-passing kernel from the committed ncu
    summary of this workload and these flags (profiles/*.md), or None when there is
    none or the kernel source has changed since the counters were taken."""
    import glob
    import hashlib
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        fields = {}
        for line in open(path):
            if ":" in line and not line.startswith(("|", "#", " ")):
                k, _, v = line.partition(":")
                fields[k.strip()] = v.strip()
        if fields.get("workload") != workload or "traffic_bytes_per_launch" not in fields:
            continue
        if int(fields.get("flags", "0")) != flags:
            continue
        src = os.path.join(ROOT, fields.get("kernel_source", ""))
        if not os.path.isfile(src):
            continue
        sha = hashlib.sha1(open(src, "rb").read()).hexdigest()[:12]
        if sha == fields.get("kernel_source_sha1_12"):
            return int(fields["traffic_bytes_per_launch"]), os.path.basename(path)
    return None, None


# ------------------------------------------------------------ CPU checker ---

def time_oracle(cfg, budget_s: float, threads: int):
    """Runs the CPU checker's whole path on `cfg` repeatedly for about
    budget_s seconds; returns (evaluations/s, seconds per pass, passes)."""
    from oracle import oracle
    oracle.build()
    oracle.forward(cfg, threads=threads, states=np.arange(min(4, cfg["B"])))   # load + warm
    t0 = time.perf_counter()
    passes = 0
    while True:
        oracle.forward(cfg, threads=threads)
        passes += 1
        el = time.perf_counter() - t0
        if el >= budget_s:
            break
    return cfg["B"] * passes / el, el / passes, passes


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg = make_workload(args.workload)
    cores = len(os.sched_getaffinity(0))
    from oracle import oracle
    oracle.build()
    steps, warmup = max(1, args.steps), max(1, args.warmup)
    sample = cfg
    # Bound the sample of states per step so that the whole run stays near two
    # minutes: time a probe of one state per core, then size the sample.
    probe = np.arange(min(cfg["B"], cores))
    oracle.forward(cfg, threads=cores, states=probe)
    t0 = time.perf_counter()
    oracle.forward(cfg, threads=cores, states=probe)
    per_state = (time.perf_counter() - t0) / len(probe)
    keep = int(120.0 / (steps + warmup) / max(per_state, 1e-9))
    keep = max(min(cores, cfg["B"]), min(cfg["B"], keep))
    states_sel = None if keep >= cfg["B"] else np.arange(keep)
    sample_desc = ("full batch of %d states per step" % cfg["B"] if states_sel is None
                   else "first %d of %d states per step" % (keep, cfg["B"]))
    nstates = cfg["B"] if states_sel is None else len(states_sel)
    for _ in range(warmup):
        oracle.forward(sample, threads=cores, states=states_sel)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.forward(sample, threads=cores, states=states_sel)
    el = time.perf_counter() - t0
    value = nstates * steps / el
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * el / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample_desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------- clocks ----

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while running."""

    def __init__(self, index: int, uuid: str | None = None):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------ B200 ----

def error_against_checker(cfg, logits, Hd, Hu, samples: int = 16):
    """The library's outputs against the CPU checker on evenly spaced states:
    elementwise error with the floor at 0.1 and at 0.01 of the row's largest
    entry, normwise error, and decisive states whose argmax differs."""
    from oracle import oracle
    B = cfg["B"]
    sel = np.arange(B) if B <= samples else np.unique(np.linspace(0, B - 1, samples).astype(int))
    ref = oracle.forward(cfg, threads=len(os.sched_getaffinity(0)), states=sel)

    def err(got, want, floor):
        row = np.max(np.abs(want), axis=-1, keepdims=True)
        den = np.maximum(np.abs(want), floor * row)
        den = np.where(den == 0, 1.0, den)
        return float(np.max(np.abs(got.astype(np.float64) - want) / den))

    got = {"H_down": Hd[:, sel].cpu().numpy(), "H_up": Hu[:, sel].cpu().numpy(), "logits": logits[sel].cpu().numpy()}
    srt = np.sort(ref["logits"], axis=1)
    gap = srt[:, -1] - srt[:, -2] if srt.shape[1] > 1 else np.full(len(srt), np.inf)
    decisive = gap > np.maximum(1e-3, 2e-5 * np.abs(ref["logits"]).max(axis=1))
    differ = got["logits"].argmax(axis=1) != ref["logits"].argmax(axis=1)
    return {"states_checked": int(len(sel)),
            "max_rel_err": max(err(got[k], ref[k], 0.1) for k in got),
            "max_rel_err_floor_0p01": max(err(got[k], ref[k], 0.01) for k in got),
            "max_norm_err": max(err(got[k], ref[k], 1.0) for k in got),
            "argmax_mismatches": int((differ & decisive).sum()), "decisive_states": int(decisive.sum()),
            "reference": "fp64 CPU checker (oracle/), same seeded inputs"}


def measure_workload(name: str, steps: int, warmup: int, flags: int, sm_count: int, peak_tflops: float):
    """Short measurement of one workload on the current device: whole path and
    the message-passing launch alone, L2 flushed before every timed call."""
    import torch
    import paper_1906_08879_b200 as placeto
    cfg = make_workload(name)
    n, B, m, d, F = cfg["n"], cfg["B"], cfg["m"], cfg["d"], cfg["F"]
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    dev_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    cost, nbytes = dev_t(cfg["cost"]), dev_t(cfg["bytes"])
    devs, cur, placed = dev_t(cfg["dev"]), dev_t(cfg["cur"]), dev_t(cfg["placed"])
    logits = torch.empty((B, m), dtype=torch.float32, device="cuda")
    probs = torch.empty((B, m), dtype=torch.float32, device="cuda")
    ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD, flags)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    X = placeto.placeto_build_features(g, cost, nbytes, devs, cur, placed, m)
    Hd = torch.empty((n, B, d), dtype=torch.float32, device="cuda")
    Hu = torch.empty((n, B, d), dtype=torch.float32, device="cuda")

    def timed(fn):
        for _ in range(warmup):
            fn()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(steps):
            flush.zero_()
            starts[i].record(stream)
            fn()
            ends[i].record(stream)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in zip(starts, ends)) / steps

    step_ms = timed(lambda: placeto.placeto_policy_forward(g, w, cost, nbytes, devs, cur, placed, logits, probs,
                                                           ws, flags, stream))
    embed_ms = timed(lambda: placeto.placeto_embed_forward(g, w, X, Hd, Hu, ws, flags, stream))
    achieved = flops_embed(cfg) / (embed_ms * 1e-3) / 1e12
    out = {"n_nodes": n, "depth": cfg["depth"], "d": d, "states": B, "ms_per_step": step_ms,
           "value": B / (step_ms * 1e-3), "embed_ms": embed_ms,
           "roofline_frac": achieved / peak_tflops if d >= 32 else None}
    out.update(error_against_checker(cfg, logits, Hd, Hu))
    del out["reference"]
    return out


def run_b200(args):
    import torch
    import paper_1906_08879_b200 as placeto

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = make_workload(args.workload, rank)
    if args.episodes > 0:   # E states per policy evaluation: the current states of the E episodes
        from gen import states as gen_states
        rng_e = np.random.Generator(np.random.PCG64(4242 + rank))
        cfg["dev"], cfg["cur"], cfg["placed"] = gen_states.random_states(rng_e, cfg["n"], cfg["m"], args.episodes)
        cfg["B"] = args.episodes
    n, B, m, d, F = cfg["n"], cfg["B"], cfg["m"], cfg["d"], cfg["F"]
    units = B * n if args.episodes > 0 else B      # policy evaluations per step
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    dev_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    cost, nbytes = dev_t(cfg["cost"]), dev_t(cfg["bytes"])
    devs, cur, placed = dev_t(cfg["dev"]), dev_t(cfg["cur"]), dev_t(cfg["placed"])
    logits = torch.empty((B, m), dtype=torch.float32, device="cuda")
    probs = torch.empty((B, m), dtype=torch.float32, device="cuda")
    ws = placeto.workspace(g, w, B, placeto.CALL_FORWARD_HOST, args.flags)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    if args.episodes > 0:
        from gen import graphs as gen_graphs
        order = dev_t(gen_graphs.topological_order(n, cfg["src"], cfg["dst"]))
        uniforms = dev_t(rng_e.random(size=(B, n)).astype(np.float32))
        dev0 = devs.clone()
        actions = torch.empty((B, n), dtype=torch.uint8, device="cuda")
        logp = torch.empty((B, n), dtype=torch.float32, device="cuda")
        ws_ep = placeto.workspace(g, w, B, placeto.CALL_EPISODE, args.flags)

    def step():
        if args.episodes > 0:
            devs.copy_(dev0)
            placeto.placeto_episode_rollout(g, w, cost, nbytes, order, devs, uniforms, actions, logp,
                                            ws_ep, args.flags, stream)
            return
        placeto.placeto_policy_forward(g, w, cost, nbytes, devs, cur, placed, logits, probs, ws,
                                       args.flags, stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, count_launches=False):
        """Sum of per-step CUDA-event times (ms) on the launching stream; L2 is
        flushed before every step, outside the events."""
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        launches = 0
        for i in range(steps):
            flush.zero_()
            starts[i].record(stream)
            fn()
            ends[i].record(stream)
            if count_launches:
                launches += placeto.placeto_last_launch_count()
        torch.cuda.synchronize()
        return sum(s.elapsed_time(e) for s, e in zip(starts, ends)), launches

    warmup = max(args.warmup, 3)
    sampler = ClockSampler(local, str(getattr(torch.cuda.get_device_properties(local), "uuid", "")))
    for _ in range(warmup):
        step()
    barrier()
    sampler.start()
    total_ms, launches = timed(step, args.steps, count_launches=True)
    barrier()
    clocks = sampler.stop()
    value, total_ms = job_throughput(total_ms, units, args.steps, dist, "cuda")

    # end to end through the host-buffer entry point: pinned inputs -> device -> results on host
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = [pin(cfg[k]) for k in ("cost", "bytes", "dev", "cur", "placed")]
    h_logits = torch.empty((B, m), dtype=torch.float32).pin_memory()
    h_probs = torch.empty((B, m), dtype=torch.float32).pin_memory()

    if args.episodes > 0:
        h_dev0 = pin(cfg["dev"])
        h_actions = torch.empty((B, n), dtype=torch.uint8).pin_memory()
        h_logp = torch.empty((B, n), dtype=torch.float32).pin_memory()

    def e2e_step():
        if args.episodes > 0:   # initial placement in, actions and log-probabilities out
            devs.copy_(h_dev0, non_blocking=True)
            placeto.placeto_episode_rollout(g, w, cost, nbytes, order, devs, uniforms, actions, logp,
                                            ws_ep, args.flags, stream)
            h_actions.copy_(actions, non_blocking=True)
            h_logp.copy_(logp, non_blocking=True)
            stream.synchronize()
            return
        placeto.placeto_policy_forward_host(g, w, *h_in, h_logits, h_probs, ws, args.flags, stream)

    for _ in range(3):
        e2e_step()
    barrier()
    e2e_ms, _ = timed(e2e_step, args.steps)
    barrier()
    e2e_value, _ = job_throughput(e2e_ms, units, args.steps, dist, "cuda")
    h2d = sum(x.numel() * x.element_size() for x in h_in)
    d2h = h_logits.numel() * 4 + h_probs.numel() * 4
    if args.episodes > 0:
        h2d, d2h = h_dev0.numel(), h_actions.numel() + 4 * h_logp.numel()
        assert torch.equal(h_actions.cuda(), actions), "host copy of the actions differs"
    else:
        assert torch.equal(h_logits.cuda(), logits), "host and device entry points disagree"

    # the dominant kernel alone: the message-passing launch(es) of embed_forward
    X = placeto.placeto_build_features(g, cost, nbytes, devs, cur, placed, m)
    Hd = torch.empty((n, B, d), dtype=torch.float32, device="cuda")
    Hu = torch.empty((n, B, d), dtype=torch.float32, device="cuda")

    ws_rounds = placeto.workspace(g, w, B, placeto.CALL_EMBED_ROUNDS) if args.rounds > 0 else None

    def embed_only():
        if args.rounds > 0:
            placeto.placeto_embed_rounds(g, w, X, args.rounds, Hd, Hu, ws_rounds, stream)
            return
        placeto.placeto_embed_forward(g, w, X, Hd, Hu, ws, args.flags, stream)

    def pool_only():
        placeto.placeto_policy_logits(g, w, X, Hd, Hu, cur, logits, probs, ws, args.flags, stream)

    for _ in range(3):
        embed_only(); pool_only()
    ksteps = min(args.steps, 100)
    embed_ms, _ = timed(embed_only, ksteps)
    embed_launches = placeto.placeto_last_launch_count()
    pool_ms, _ = timed(pool_only, ksteps)
    embed_ms /= ksteps
    pool_ms /= ksteps

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    sm_count = torch.cuda.get_device_properties(0).multi_processor_count
    sm_max_mhz = clocks["sm_max_mhz"] or 1965
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        sm_max_mhz = json.load(open(peaks_path)).get("sm_max_mhz", sm_max_mhz)
    hbm_peak, hbm_src = 6650.0, "fallback (earlier measurement on this pool)"
    if os.path.exists(peaks_path):
        hbm_peak = float(json.load(open(peaks_path)).get("hbm_gbs", hbm_peak))
        hbm_src = "measured (MEASURED_PEAKS.json)"
    peak_tflops = sm_count * FP32_LANES_PER_SM * 2 * sm_max_mhz * 1e6 / 1e12
    achieved = flops_embed(cfg) * max(1, args.rounds) / (embed_ms * 1e-3) / 1e12
    traffic, traffic_from = measured_traffic(cfg["name"], args.flags)
    roofline = {"bound": "alu",
                "kernel": ("message passing (embed_rounds, %d synchronous rounds, %d launches)" % (args.rounds, embed_launches)
                           if args.rounds > 0 else "message passing (embed_forward, %d launch(es))" % embed_launches),
                "achieved": achieved, "peak": peak_tflops, "unit": "TFLOP/s", "frac": achieved / peak_tflops,
                "traffic": traffic, "traffic_source": traffic_from,
                "arithmetic": ("fp32 accumulate on tcgen05.mma, TF32 head+tail operands (4 products per instruction)"
                               if d == 64 and (args.flags & 64) and not (args.flags & 24)
                               else "fp32 accumulate on mma.sync, TF32 head+tail operands (3 products)"
                               if d == 64 and not (args.flags & 24) else "fp32 fma"),
                "algorithmic_bytes": (4 * F + 8 * d) * n * B,
                "hbm": {"achieved": (4 * F + 8 * d) * n * B / (embed_ms * 1e-3) / 1e9, "peak": hbm_peak,
                        "unit": "GB/s", "frac": (4 * F + 8 * d) * n * B / (embed_ms * 1e-3) / 1e9 / hbm_peak,
                        "peak_source": hbm_src},
                "peak_source": "derived: %d SMs x 128 FP32 FMA lanes x 2 flop x %.0f MHz max SM clock"
                               % (sm_count, sm_max_mhz),
                "ms_per_launch": embed_ms,
                "pooling_head_ms": pool_ms,
                "pooling_achieved_tflops": flops_pool(cfg) / (pool_ms * 1e-3) / 1e12}

    cores = len(os.sched_getaffinity(0))
    cpu_value, cpu_s, passes = time_oracle(cfg, args.cpu_baseline_seconds, cores)
    config = workload_config(cfg, world)
    parity = None
    others = None
    if args.episodes == 0:
        step()                                        # the outputs of this rank's own batch
        embed_only()
        torch.cuda.synchronize()
        parity = error_against_checker(cfg, logits, Hd, Hu)
        if world == 1 and not args.no_others and args.rounds == 0:
            others = {}
            for other in ("tiny", "inception", "nmt", "sweep63", "nasnet_wide", "nasnet"):
                if other != cfg["name"] and not (other == "sweep63" and cfg["name"].startswith("sweep")):
                    others[other] = measure_workload(other, min(args.steps, 30), 3, args.flags, sm_count, peak_tflops)
    if args.episodes > 0:
        config.update(workload=cfg["name"] + "-episodes", episodes_per_gpu=B, steps_per_episode=n,
                      choice="sampled (inverse CDF of the device softmax)",
                      l2="flushed between timed rollouts only (256 MiB memset, outside the timed events)")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches, "roofline": roofline,
            "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "%d full passes over the batch of %d states (%.2f s each)"
                                       % (passes, B, cpu_s)}}
    if parity is not None:
        line["parity"] = parity
        for k in ("max_rel_err", "max_norm_err", "argmax_mismatches"):
            line[k] = parity[k]
    if others is not None:
        line["other_workloads"] = others
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_simulator(args):
    """Extra mode: the runtime simulator on P random placements (one JSON line, own metric)."""
    import torch
    import paper_1906_08879_b200 as placeto
    from oracle import simulator
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    cfg = make_workload(args.workload)
    n, m, P = cfg["n"], cfg["m"], args.simulate
    rng = np.random.Generator(np.random.PCG64(99))
    devs_h = rng.integers(0, m, size=(P, n)).astype(np.uint8)
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    dev_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    cost, nbytes, devs = dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(devs_h)
    out = torch.empty((P,), dtype=torch.float64, device="cuda")
    bw = 1e4
    need = int(placeto.binding._lib.placeto_simulator_workspace_bytes(g.handle, P, m))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        placeto.placeto_simulate_runtime(g, cost, nbytes, devs, m, bw, out, ws, stream)
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record(stream)
    for _ in range(args.steps):
        placeto.placeto_simulate_runtime(g, cost, nbytes, devs, m, bw, out, ws, stream)
    e.record(stream)
    torch.cuda.synchronize()
    ms = s.elapsed_time(e) / args.steps
    k = min(P, 32)
    t0 = time.perf_counter()
    ref = simulator.runtimes(n, cfg["src"], cfg["dst"], cfg["cost"], cfg["bytes"], devs_h[:k], m, bw)
    cpu_s = time.perf_counter() - t0
    assert np.array_equal(out.cpu().numpy()[:k], ref), "simulator disagrees with the CPU checker"
    print(json.dumps({"metric": "simulated placements/sec (event-based runtime simulator)",
                      "value": P / (ms * 1e-3), "unit": "placements/s", "n_gpus": 1, "steps": args.steps,
                      "ms_per_step": ms, "higher_is_better": True, "dtype": "f64", "data": "synthetic",
                      "config": {"workload": cfg["name"] + "-simulator", "n_nodes": n, "placements": P,
                                 "devices": m, "bandwidth": bw},
                      "cpu_baseline": {"value": k / cpu_s, "unit": "placements/s", "cores": 1, "kind": "oracle",
                                       "sample": "%d placements, pure-Python event loop" % k}}))
    return 0


def run_gradient(args):
    """Extra mode: the policy gradient of one batch (forward intermediates X, H given)."""
    import torch
    import paper_1906_08879_b200 as placeto
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    cfg = make_workload(args.workload)
    n, B, m = cfg["n"], cfg["B"], cfg["m"]
    g = placeto.Graph(n, cfg["src"], cfg["dst"])
    w = placeto.Weights(cfg["weights"])
    dev_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    cur = dev_t(cfg["cur"])
    X = placeto.placeto_build_features(g, dev_t(cfg["cost"]), dev_t(cfg["bytes"]), dev_t(cfg["dev"]), cur,
                                       dev_t(cfg["placed"]), m)
    Hd, Hu = placeto.placeto_embed_forward(g, w, X)
    rng = np.random.Generator(np.random.PCG64(7))
    actions = dev_t(rng.integers(0, m, B).astype(np.int32))
    adv = dev_t(rng.normal(size=B).astype(np.float32))
    grads = placeto.binding.zero_gradients(cfg["weights"])
    ws = placeto.workspace(g, w, B, placeto.CALL_GRADIENT)
    stream = torch.cuda.current_stream()
    run = lambda: placeto.placeto_policy_gradient(g, w, X, Hd, Hu, cur, actions, adv, 0.01, grads, ws, stream)
    for _ in range(max(args.warmup, 3)):
        run()
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record(stream)
    for _ in range(args.steps):
        run()
    e.record(stream)
    torch.cuda.synchronize()
    ms = s.elapsed_time(e) / args.steps
    d, F = cfg["d"], cfg["F"]
    flop = 3.0 * (flops_embed(cfg) + flops_pool(cfg))      # recompute + two products per forward product
    print(json.dumps({"metric": "states differentiated/sec (policy gradient, embeddings given)",
                      "value": B / (ms * 1e-3), "unit": "states/s", "n_gpus": 1, "steps": args.steps,
                      "ms_per_step": ms, "higher_is_better": True, "dtype": "f32", "data": "synthetic",
                      "gpu_launches": placeto.placeto_last_launch_count(),
                      "config": {"workload": cfg["name"] + "-gradient", "n_nodes": n, "states": B, "d": d, "F": F,
                                 "workspace_bytes": int(ws.numel())},
                      "approx_tflops": flop / (ms * 1e-3) / 1e12}))
    return 0


def main():
    args = parse_args()
    if args.gradient and args.impl != "reference":
        return run_gradient(args)
    if args.simulate > 0 and args.impl != "reference":
        return run_simulator(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_b200(args)


if __name__ == "__main__":
    sys.exit(main())
