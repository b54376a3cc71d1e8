"""Thin ctypes binding of libplaceto.so (see include/placeto.h).

Argument marshalling only: every step of the policy forward runs in the CUDA
library. PyTorch supplies device memory and streams. The functions carry the
names of the C entry points; tensors must live on the CUDA device that was
current when the graph was created. If the shared library is missing the
import fails loudly: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PLACETO_LIBRARY=debug selects the build whose kernels check their indices (build.py --debug),
# PLACETO_LIBRARY=timers the one whose tcgen05 kernels print phase timers (build.py --timers)
LIB_PATH = os.path.join(_HERE, {"debug": "libplaceto_debug.so", "timers": "libplaceto_timers.so"}.get(
    os.environ.get("PLACETO_LIBRARY", ""), "libplaceto.so"))

# flags and enums of placeto.h
PLACETO_AUTO, PLACETO_PER_LEVEL, PLACETO_SLICED, PLACETO_COOPERATIVE, PLACETO_GENERIC = 0, 1, 2, 4, 8
PLACETO_FMA_ONLY, PLACETO_TENSOR, PLACETO_TCGEN05, PLACETO_PIPELINE = 16, 32, 64, 128
PLACETO_GRAPH_DEVICE, PLACETO_GRAPH_HOST_ONLY = 0, 1
CALL_EMBED, CALL_LOGITS, CALL_FORWARD, CALL_FORWARD_HOST, CALL_EPISODE, CALL_EMBED_ROUNDS, CALL_GRADIENT = 0, 1, 2, 3, 4, 5, 6

EXPORTS = (
    "placeto_status_string", "placeto_graph_create", "placeto_graph_info",
    "placeto_graph_host_view", "placeto_graph_destroy", "placeto_workspace_bytes",
    "placeto_build_features", "placeto_embed_forward", "placeto_policy_logits",
    "placeto_policy_forward", "placeto_policy_forward_host", "placeto_policy_logits_static",
    "placeto_episode_rollout", "placeto_embed_rounds", "placeto_simulator_workspace_bytes", "placeto_simulate_runtime",
    "placeto_policy_gradient", "placeto_last_launch_count", "placeto_last_status", "placeto_debug_wait_timeout",
    "placeto_simple_aggregator", "placeto_simulate_placements",
)


class PlacetoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class _Mlp(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("in_dim", ctypes.c_int32),
                ("hidden_dim", ctypes.c_int32), ("out_dim", ctypes.c_int32),
                ("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p),
                ("W2", ctypes.c_void_p), ("b2", ctypes.c_void_p),
                ("act", ctypes.c_int32), ("final_act", ctypes.c_int32)]


class _Weights(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("F", ctypes.c_int32), ("m", ctypes.c_int32),
                ("f_down", _Mlp), ("g_down", _Mlp), ("f_up", _Mlp), ("g_up", _Mlp),
                ("l", _Mlp * 3), ("h", _Mlp * 3), ("head", _Mlp)]


class _AggWeights(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("F", ctypes.c_int32), ("m", ctypes.c_int32),
                ("l", _Mlp), ("h", _Mlp), ("head", _Mlp)]


class _LevelView(ctypes.Structure):
    _fields_ = [("n_levels", ctypes.c_int32), ("level_ptr", ctypes.POINTER(ctypes.c_int32)),
                ("order", ctypes.POINTER(ctypes.c_int32)), ("nbr_ptr", ctypes.POINTER(ctypes.c_int32)),
                ("nbr", ctypes.POINTER(ctypes.c_int32)), ("n_slots", ctypes.c_int32),
                ("own_slot", ctypes.POINTER(ctypes.c_int32)),
                ("nbr_slot", ctypes.POINTER(ctypes.c_int32))]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libplaceto.so is missing (%s): build it with "
            "`python paper_1906_08879_b200/build.py`; there is no CPU fallback" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    lib.placeto_status_string.restype = ctypes.c_char_p
    lib.placeto_status_string.argtypes = [ctypes.c_int]
    lib.placeto_graph_destroy.restype = None
    lib.placeto_graph_destroy.argtypes = [ctypes.c_void_p]
    lib.placeto_workspace_bytes.restype = ctypes.c_size_t
    lib.placeto_last_launch_count.restype = ctypes.c_int32
    lib.placeto_simulator_workspace_bytes.restype = ctypes.c_size_t
    for name in ("placeto_graph_create", "placeto_graph_info", "placeto_graph_host_view",
                 "placeto_build_features", "placeto_embed_forward", "placeto_policy_logits",
                 "placeto_policy_forward", "placeto_policy_forward_host",
                 "placeto_policy_logits_static", "placeto_episode_rollout", "placeto_embed_rounds", "placeto_simulate_runtime", "placeto_policy_gradient",
                 "placeto_last_status", "placeto_debug_wait_timeout", "placeto_simple_aggregator",
                 "placeto_simulate_placements"):
        getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.placeto_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise PlacetoError(status, where)


def _p(t):
    """Device (or host) address of a tensor / numpy array, or NULL."""
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, np.ndarray):
        return ctypes.c_void_p(t.ctypes.data)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Graph:
    """Owner of a placeto_graph handle."""

    def __init__(self, n: int, src, dst, host_only: bool = False):
        src = np.ascontiguousarray(src, dtype=np.int32)
        dst = np.ascontiguousarray(dst, dtype=np.int32)
        if src.shape != dst.shape or src.ndim != 1:
            raise ValueError("src and dst must be 1-D arrays of equal length")
        self._h = ctypes.c_void_p(0)
        self.n = int(n)
        self.host_only = host_only
        _check(_lib.placeto_graph_create(
            ctypes.c_int32(n), ctypes.c_int64(len(src)), _p(src) if len(src) else None,
            _p(dst) if len(dst) else None,
            ctypes.c_uint32(PLACETO_GRAPH_HOST_ONLY if host_only else PLACETO_GRAPH_DEVICE),
            ctypes.byref(self._h)), "placeto_graph_create")

    @property
    def handle(self):
        return self._h

    def info(self) -> dict:
        n, ne = ctypes.c_int32(), ctypes.c_int64()
        ld, lu, mw = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(_lib.placeto_graph_info(self._h, ctypes.byref(n), ctypes.byref(ne), ctypes.byref(ld),
                                       ctypes.byref(lu), ctypes.byref(mw)), "placeto_graph_info")
        return {"n": n.value, "n_edges": ne.value, "n_levels_down": ld.value,
                "n_levels_up": lu.value, "max_level_width": mw.value}

    def host_view(self) -> dict:
        """Copies of the host plan as numpy arrays (for inspection and tests)."""
        down, up = _LevelView(), _LevelView()
        rel = ctypes.POINTER(ctypes.c_uint8)()
        _check(_lib.placeto_graph_host_view(self._h, ctypes.byref(down), ctypes.byref(up),
                                            ctypes.byref(rel)), "placeto_graph_host_view")
        n = self.n
        out = {}
        for name, v in (("down", down), ("up", up)):
            nbr_ptr = np.ctypeslib.as_array(v.nbr_ptr, shape=(n + 1,)).copy()
            out[name] = {
                "n_levels": v.n_levels,
                "level_ptr": np.ctypeslib.as_array(v.level_ptr, shape=(v.n_levels + 1,)).copy(),
                "order": np.ctypeslib.as_array(v.order, shape=(n,)).copy(),
                "nbr_ptr": nbr_ptr,
                "nbr": (np.ctypeslib.as_array(v.nbr, shape=(int(nbr_ptr[-1]),)).copy()
                        if nbr_ptr[-1] > 0 else np.zeros(0, np.int32)),
                "n_slots": v.n_slots,
                "own_slot": np.ctypeslib.as_array(v.own_slot, shape=(n,)).copy(),
                "nbr_slot": (np.ctypeslib.as_array(v.nbr_slot, shape=(int(nbr_ptr[-1]),)).copy()
                             if nbr_ptr[-1] > 0 else np.zeros(0, np.int32)),
            }
        out["relation"] = np.ctypeslib.as_array(rel, shape=(n, n)).copy()
        return out

    def close(self) -> None:
        if self._h:
            _lib.placeto_graph_destroy(self._h)
            self._h = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Weights:
    """Device copies of the policy's networks and the C struct that points at
    them. Built from the dict layout of gen.states.policy_weights (numpy
    arrays W[in][out], biases, layer counts, activation switches)."""

    def __init__(self, weights: dict, device="cuda"):
        self.d, self.F, self.m = int(weights["d"]), int(weights["F"]), int(weights["m"])
        self._keep = []
        self.tensors = {}            # (net name, index or None, array name) -> device tensor
        self.c = _Weights()
        self.c.d, self.c.F, self.c.m = self.d, self.F, self.m
        dev = torch.device(device)
        for name in ("f_down", "g_down", "f_up", "g_up", "head"):
            if name in weights:
                setattr(self.c, name, self._mlp(weights[name], dev, (name, None)))
        for name in ("l", "h"):
            if name in weights:
                arr = getattr(self.c, name)
                for i in range(3):
                    arr[i] = self._mlp(weights[name][i], dev, (name, i))

    def _mlp(self, net: dict, dev, where=None) -> _Mlp:
        ptr = {}
        for k in ("W1", "b1", "W2", "b2"):
            a = net.get(k)
            if a is None:
                ptr[k] = None
                continue
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev)
            self._keep.append(t)
            if where is not None:
                self.tensors[where + (k,)] = t
            ptr[k] = t.data_ptr()
        return _Mlp(net["n_layers"], net["in_dim"], net.get("hidden_dim", net["out_dim"]),
                    net["out_dim"], ptr["W1"], ptr["b1"], ptr["W2"], ptr["b2"],
                    net["act"], net["final_act"])


def placeto_workspace_bytes(g: Graph, w: Weights, B: int, call: int, flags: int = 0) -> int:
    return int(_lib.placeto_workspace_bytes(g.handle, ctypes.byref(w.c), ctypes.c_int32(B),
                                            ctypes.c_int(call), ctypes.c_uint32(flags)))


def workspace(g: Graph, w: Weights, B: int, call: int, flags: int = 0, device="cuda"):
    """Allocates a workspace tensor of the size the call needs."""
    nbytes = placeto_workspace_bytes(g, w, B, call, flags)
    if nbytes == 0:
        raise PlacetoError(1, "placeto_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def placeto_build_features(g: Graph, cost, nbytes, dev, cur, placed, m: int, X=None, stream=None):
    B = dev.shape[0]
    if X is None:
        X = torch.empty((g.n, B, m + 4), dtype=torch.float32, device=dev.device)
    _check(_lib.placeto_build_features(g.handle, _p(cost), _p(nbytes), _p(dev), _p(cur), _p(placed),
                                       ctypes.c_int32(m), ctypes.c_int32(B), _p(X), _stream(stream)),
           "placeto_build_features")
    return X


def placeto_embed_forward(g: Graph, w: Weights, X, H_down=None, H_up=None, ws=None,
                          flags: int = 0, stream=None):
    B = X.shape[1]
    if H_down is None:
        H_down = torch.empty((g.n, B, w.d), dtype=torch.float32, device=X.device)
    if H_up is None:
        H_up = torch.empty((g.n, B, w.d), dtype=torch.float32, device=X.device)
    if ws is None:
        ws = workspace(g, w, B, CALL_EMBED, flags, X.device)
    _check(_lib.placeto_embed_forward(g.handle, ctypes.byref(w.c), _p(X), ctypes.c_int32(B),
                                      _p(H_down), _p(H_up), _p(ws), ctypes.c_size_t(ws.numel()),
                                      ctypes.c_uint32(flags), _stream(stream)),
           "placeto_embed_forward")
    return H_down, H_up


def placeto_embed_rounds(g: Graph, w: Weights, X, rounds: int, H_down=None, H_up=None, ws=None,
                         stream=None):
    """The synchronous k-round form of the message passing (from zeros)."""
    B = X.shape[1]
    if H_down is None:
        H_down = torch.empty((g.n, B, w.d), dtype=torch.float32, device=X.device)
    if H_up is None:
        H_up = torch.empty((g.n, B, w.d), dtype=torch.float32, device=X.device)
    if ws is None:
        ws = workspace(g, w, B, CALL_EMBED_ROUNDS, 0, X.device)
    _check(_lib.placeto_embed_rounds(g.handle, ctypes.byref(w.c), _p(X), ctypes.c_int32(B),
                                     ctypes.c_int32(rounds), _p(H_down), _p(H_up), _p(ws),
                                     ctypes.c_size_t(ws.numel()), _stream(stream)),
           "placeto_embed_rounds")
    return H_down, H_up


def placeto_policy_logits(g: Graph, w: Weights, X, H_down, H_up, cur, logits=None, probs=None,
                          ws=None, flags: int = 0, stream=None, want_probs: bool = True):
    B = X.shape[1]
    if logits is None:
        logits = torch.empty((B, w.m), dtype=torch.float32, device=X.device)
    if probs is None and want_probs:
        probs = torch.empty((B, w.m), dtype=torch.float32, device=X.device)
    if ws is None:
        ws = workspace(g, w, B, CALL_LOGITS, flags, X.device)
    _check(_lib.placeto_policy_logits(g.handle, ctypes.byref(w.c), _p(X), _p(H_down), _p(H_up),
                                      _p(cur), ctypes.c_int32(B), _p(logits), _p(probs), _p(ws),
                                      ctypes.c_size_t(ws.numel()), ctypes.c_uint32(flags),
                                      _stream(stream)), "placeto_policy_logits")
    return logits, probs


def placeto_policy_forward(g: Graph, w: Weights, cost, nbytes, dev, cur, placed, logits=None,
                           probs=None, ws=None, flags: int = 0, stream=None):
    B = dev.shape[0]
    if logits is None:
        logits = torch.empty((B, w.m), dtype=torch.float32, device=dev.device)
    if probs is None:
        probs = torch.empty((B, w.m), dtype=torch.float32, device=dev.device)
    if ws is None:
        ws = workspace(g, w, B, CALL_FORWARD, flags, dev.device)
    _check(_lib.placeto_policy_forward(g.handle, ctypes.byref(w.c), _p(cost), _p(nbytes), _p(dev),
                                       _p(cur), _p(placed), ctypes.c_int32(B), _p(logits), _p(probs),
                                       _p(ws), ctypes.c_size_t(ws.numel()), ctypes.c_uint32(flags),
                                       _stream(stream)), "placeto_policy_forward")
    return logits, probs


def placeto_policy_forward_host(g: Graph, w: Weights, cost, nbytes, dev, cur, placed, logits,
                                probs, ws, flags: int = 0, stream=None):
    """All state arrays and results are HOST buffers (numpy arrays or CPU
    tensors, ideally pinned); `ws` is a device workspace sized for
    CALL_FORWARD_HOST. Returns after the results have arrived."""
    B = dev.shape[0]
    _check(_lib.placeto_policy_forward_host(g.handle, ctypes.byref(w.c), _p(cost), _p(nbytes),
                                            _p(dev), _p(cur), _p(placed), ctypes.c_int32(B),
                                            _p(logits), _p(probs), _p(ws),
                                            ctypes.c_size_t(ws.numel()), ctypes.c_uint32(flags),
                                            _stream(stream)), "placeto_policy_forward_host")
    return logits, probs


STATIC_SCRATCH_BYTES = 4 << 20


def placeto_policy_logits_static(g: Graph, w: Weights, X, H_down, H_up, cur, logits, probs=None,
                                 flags: int = 0, stream=None):
    """placeto_policy_logits for callers that may not allocate device memory:
    no workspace argument, the chunk partial sums live in an array built into
    the library (STATIC_SCRATCH_BYTES per GPU). This wrapper allocates nothing
    either, so `logits` (and `probs`, if wanted) must be passed in. Raises
    PlacetoError with status 7 when the batch needs more scratch than the array
    holds. Calls on one device share that array: do not let two overlap."""
    B = X.shape[1]
    _check(_lib.placeto_policy_logits_static(g.handle, ctypes.byref(w.c), _p(X), _p(H_down),
                                             _p(H_up), _p(cur), ctypes.c_int32(B), _p(logits),
                                             _p(probs), ctypes.c_uint32(flags), _stream(stream)),
           "placeto_policy_logits_static")
    return logits, probs


def placeto_episode_rollout(g: Graph, w: Weights, cost, nbytes, order, dev, uniforms=None,
                            actions=None, logp=None, ws=None, flags: int = 0, stream=None):
    """E = dev.shape[0] episodes over the graph; `dev` (uint8 [E][n]) holds the
    initial placement and is overwritten with the final one. `uniforms` (float
    [E][n]) switches from greedy to sampled choices. Returns (dev, actions, logp)."""
    E = dev.shape[0]
    if actions is None:
        actions = torch.empty((E, g.n), dtype=torch.uint8, device=dev.device)
    if logp is None:
        logp = torch.empty((E, g.n), dtype=torch.float32, device=dev.device)
    if ws is None:
        ws = workspace(g, w, E, CALL_EPISODE, flags, dev.device)
    _check(_lib.placeto_episode_rollout(g.handle, ctypes.byref(w.c), _p(cost), _p(nbytes), _p(order),
                                        _p(uniforms), ctypes.c_int32(E), _p(dev), _p(actions),
                                        _p(logp), _p(ws), ctypes.c_size_t(ws.numel()),
                                        ctypes.c_uint32(flags), _stream(stream)),
           "placeto_episode_rollout")
    return dev, actions, logp


def placeto_simulate_runtime(g: Graph, cost, nbytes, dev, m: int, bandwidth: float, runtime=None,
                             ws=None, stream=None):
    """Simulated run time (float64 [P]) of the P placements in `dev` (uint8 [P][n])."""
    P = dev.shape[0]
    if runtime is None:
        runtime = torch.empty((P,), dtype=torch.float64, device=dev.device)
    if ws is None:
        need = int(_lib.placeto_simulator_workspace_bytes(g.handle, ctypes.c_int32(P), ctypes.c_int32(m)))
        if need == 0:
            raise PlacetoError(1, "placeto_simulator_workspace_bytes")
        ws = torch.empty(need, dtype=torch.uint8, device=dev.device)
    _check(_lib.placeto_simulate_runtime(g.handle, _p(cost), _p(nbytes), _p(dev), ctypes.c_int32(P),
                                         ctypes.c_int32(m), ctypes.c_double(bandwidth), _p(runtime),
                                         _p(ws), ctypes.c_size_t(ws.numel()), _stream(stream)),
           "placeto_simulate_runtime")
    return runtime


def placeto_simulate_placements(g: Graph, cost, nbytes, dev, m: int, bandwidth: float, mem_limit: float,
                                mem_scale: float, ws=None, stream=None):
    """Run time [P], peak memory per device [P][m] and memory-penalised run time R(p) [P]
    (float64) of the P placements in `dev` (uint8 [P][n])."""
    P = dev.shape[0]
    runtime = torch.empty((P,), dtype=torch.float64, device=dev.device)
    peak = torch.empty((P, m), dtype=torch.float64, device=dev.device)
    pen = torch.empty((P,), dtype=torch.float64, device=dev.device)
    if ws is None:
        need = int(_lib.placeto_simulator_workspace_bytes(g.handle, ctypes.c_int32(P), ctypes.c_int32(m)))
        if need == 0:
            raise PlacetoError(1, "placeto_simulator_workspace_bytes")
        ws = torch.empty(need, dtype=torch.uint8, device=dev.device)
    _check(_lib.placeto_simulate_placements(g.handle, _p(cost), _p(nbytes), _p(dev), ctypes.c_int32(P),
                                            ctypes.c_int32(m), ctypes.c_double(bandwidth), ctypes.c_double(mem_limit),
                                            ctypes.c_double(mem_scale), _p(runtime), _p(peak), _p(pen), _p(ws),
                                            ctypes.c_size_t(ws.numel()), _stream(stream)),
           "placeto_simulate_placements")
    return runtime, peak, pen


def zero_gradients(weights: dict, device="cuda") -> "Weights":
    """A Weights object of the same shapes filled with zeros (gradient buffers)."""
    def z(net):
        out = dict(net)
        for k in ("W1", "b1", "W2", "b2"):
            if net.get(k) is not None:
                out[k] = np.zeros_like(np.asarray(net[k], dtype=np.float32))
        return out
    g = {k: weights[k] for k in ("d", "F", "m")}
    for k in ("f_down", "g_down", "f_up", "g_up", "head"):
        g[k] = z(weights[k])
    for k in ("l", "h"):
        g[k] = [z(x) for x in weights[k]]
    return Weights(g, device)


def placeto_policy_gradient(g: Graph, w: Weights, X, H_down, H_up, cur, actions, advantages,
                            beta: float, grads: Weights, ws=None, stream=None, accumulate: bool = False):
    """dJ/d(weights) into `grads` (a Weights of the same shapes, see zero_gradients);
    with `accumulate` it is added to what `grads` holds."""
    B = X.shape[1]
    if ws is None:
        ws = workspace(g, w, B, CALL_GRADIENT, 0, X.device)
    _check(_lib.placeto_policy_gradient(g.handle, ctypes.byref(w.c), _p(X), _p(H_down), _p(H_up), _p(cur),
                                        _p(actions), _p(advantages), ctypes.c_float(beta),
                                        ctypes.c_int32(B), ctypes.byref(grads.c), _p(ws),
                                        ctypes.c_size_t(ws.numel()), ctypes.c_uint32(1 if accumulate else 0),
                                        _stream(stream)),
           "placeto_policy_gradient")
    return grads


class AggregatorWeights:
    """Device copies of the simple aggregator's three networks ({"d", "F", "m", "l", "h", "head"})."""

    def __init__(self, weights: dict, device="cuda"):
        self.d, self.F, self.m = int(weights["d"]), int(weights["F"]), int(weights["m"])
        self._w = Weights({"d": self.d, "F": self.F, "m": self.m}, device)
        self.c = _AggWeights()
        self.c.d, self.c.F, self.c.m = self.d, self.F, self.m
        dev = torch.device(device)
        for name in ("l", "h", "head"):
            setattr(self.c, name, self._w._mlp(weights[name], dev))


def placeto_simple_aggregator(g: Graph, w: AggregatorWeights, X, logits=None, probs=None, stream=None):
    """The "simple aggregator" ablation: softmax(head(h(sum over all nodes of l(x_u))))."""
    B = X.shape[1]
    if logits is None:
        logits = torch.empty((B, w.m), dtype=torch.float32, device=X.device)
    if probs is None:
        probs = torch.empty((B, w.m), dtype=torch.float32, device=X.device)
    _check(_lib.placeto_simple_aggregator(g.handle, ctypes.byref(w.c), _p(X), ctypes.c_int32(B), _p(logits),
                                          _p(probs), _stream(stream)), "placeto_simple_aggregator")
    return logits, probs


def placeto_last_status(g: Graph, ws=None, stream=None) -> int:
    """Status the kernels of the latest call on `g` reported (0 = ok, 8 = a bounded wait ran
    out); synchronises the stream. `ws`: that call's workspace, None after the _static call."""
    return int(_lib.placeto_last_status(g.handle, _p(ws), _stream(stream)))


def placeto_debug_wait_timeout(g: Graph, ws, stream=None) -> None:
    """Launches the kernel whose wait is built to run out (tests of the error channel)."""
    _check(_lib.placeto_debug_wait_timeout(g.handle, _p(ws), ctypes.c_size_t(ws.numel()), _stream(stream)),
           "placeto_debug_wait_timeout")


def placeto_last_launch_count() -> int:
    return int(_lib.placeto_last_launch_count())
