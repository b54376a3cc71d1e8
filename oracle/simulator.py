"""CPU checker of the placement runtime simulator (test infrastructure only):
the event-based execution model of Appendix A.5 ("Simulator") of the Placeto
paper, written out plainly with a priority queue of events.

Model (paper): every device d has a FIFO queue of runnable operations and runs
one operation at a time; every device has a FIFO queue of output tensors to be
sent from d and its bus sends one at a time, overlapping with compute; an
operation is runnable on its device once all its parents have finished and
their outputs have arrived there; an operation takes its profiled run time, a
transfer takes size / bandwidth; the simulated run time is the time stamp of
the last Op-done event.

Readings where the paper is silent:
  * one run time per operation (the synthetic inputs carry one cost per node,
    the paper profiles each operation on each device);
  * an output tensor is sent once to each distinct device that hosts a child,
    in ascending order of the children's ids that first name that device;
  * a Wakeup of a free device or bus carries the current time stamp, so it is
    handled at once: a free device (bus) starts the head of its queue in the
    handler that filled the queue;
  * events with equal time stamps are handled in the order they were created;
  * operations without parents enter their queues in ascending id at time 0.

Peak memory (the paper: start and end time stamps of the operations, together
with the tensor sizes, predict the peak memory utilisation of the devices; it
does not say when a tensor is released). Reading: a copy of an operation's
output tensor occupies a device
  * at home (the producer's device): from the START of the producer (its output
    buffer is allocated when it begins to run) until every child placed there
    has finished AND every transfer of the tensor to other devices is done;
  * on another device that hosts a child: from the START of the transfer to that
    device (the receive buffer) until every child placed there has finished;
  * the output of an operation without children is never released (a result of
    the graph).
A device's utilisation is the sum of the copies it holds; the peak is its
maximum over the timeline; the placement's peak m is the largest peak over the
devices. The memory-penalised run time of Appendix A.7 is
    R(p) = r                     if m <= M,
           r + c * (m - M)       otherwise.
All times and byte counts are IEEE doubles; cost and size are the float32
inputs widened; sums run in event order (parents in ascending id inside one
event), so the CUDA library reproduces them bit for bit.
"""
from __future__ import annotations

import heapq
from collections import deque

import numpy as np


def children_lists(n, src, dst):
    chi = [set() for _ in range(n)]
    npar = [set() for _ in range(n)]
    for u, v in zip(map(int, src), map(int, dst)):
        chi[u].add(v)
        npar[v].add(u)
    return [sorted(c) for c in chi], [len(p) for p in npar]


def runtime(n, src, dst, cost, nbytes, dev, m, bandwidth):
    """Simulated run time of one placement. dev: device of each node (< m)."""
    return simulate(n, src, dst, cost, nbytes, dev, m, bandwidth)[0]


def penalised_runtime(r, peak, mem_limit, scale):
    """R(p) of Appendix A.7 for run time r and peak memory `peak` (largest over devices)."""
    return r if peak <= mem_limit else r + scale * (peak - mem_limit)


def simulate(n, src, dst, cost, nbytes, dev, m, bandwidth):
    """One placement: (run time, peak memory per device [m])."""
    chi, npar = children_lists(n, src, dst)
    par = [[] for _ in range(n)]
    for u in range(n):
        for c in chi[u]:
            par[c].append(u)                      # ascending u
    finished = [False] * n
    tr_left = [0] * n                            # transfers of a tensor queued or in flight
    mem = [0.0] * m
    peak = [0.0] * m

    def hold(d, o):
        mem[d] += size[o]
        if mem[d] > peak[d]:
            peak[d] = mem[d]

    def maybe_release(u, d):
        """The copy of u's output on device d, once nothing there needs it any more."""
        if not chi[u]:
            return
        if any(dev[c] == d and not finished[c] for c in chi[u]):
            return
        if d == dev[u] and tr_left[u] > 0:
            return
        mem[d] -= size[u]

    cost = [float(np.float32(c)) for c in cost]
    size = [float(np.float32(b)) for b in nbytes]
    dev = [int(d) for d in dev]
    pending = list(npar)
    q_op = [deque() for _ in range(m)]
    q_tr = [deque() for _ in range(m)]          # entries (op, destination device)
    dev_busy = [False] * m
    bus_busy = [False] * m
    events = []                                  # (time, sequence, kind, a, b)
    seq = 0
    last_op_done = 0.0

    def start_op(d, now):
        nonlocal seq
        o = q_op[d].popleft()
        dev_busy[d] = True
        hold(d, o)
        heapq.heappush(events, (now + cost[o], seq, 0, o, d))
        seq += 1

    def start_transfer(d, now):
        nonlocal seq
        o, to = q_tr[d].popleft()
        bus_busy[d] = True
        hold(to, o)
        heapq.heappush(events, (now + size[o] / bandwidth, seq, 1, o, to))
        seq += 1

    for v in range(n):
        if pending[v] == 0:
            q_op[dev[v]].append(v)
    for d in range(m):
        if q_op[d]:
            start_op(d, 0.0)
    done = 0
    while events:
        now, _, kind, o, to = heapq.heappop(events)
        if kind == 0:                            # Op-done: o finished on device `to`
            d = to
            done += 1
            last_op_done = now
            finished[o] = True
            for u in par[o]:                     # the inputs o read on its device
                maybe_release(u, d)
            sent = set()
            for c in chi[o]:
                dc = dev[c]
                if dc != d:
                    if dc not in sent:           # the tensor goes to each device once
                        sent.add(dc)
                        q_tr[d].append((o, dc))
                        tr_left[o] += 1
                else:
                    pending[c] -= 1
                    if pending[c] == 0:
                        q_op[d].append(c)
            if not bus_busy[d] and q_tr[d]:
                start_transfer(d, now)
            dev_busy[d] = False
            if q_op[d]:
                start_op(d, now)
        else:                                    # Transfer-done: o's output arrived on `to`
            d = dev[o]
            tr_left[o] -= 1
            maybe_release(o, d)
            for c in chi[o]:
                if dev[c] == to:
                    pending[c] -= 1
                    if pending[c] == 0:
                        q_op[to].append(c)
            if not dev_busy[to] and q_op[to]:
                start_op(to, now)
            bus_busy[d] = False
            if q_tr[d]:
                start_transfer(d, now)
    if done != n:
        raise ValueError("not every operation ran: the graph has a cycle")
    return last_op_done, np.asarray(peak)


def runtimes(n, src, dst, cost, nbytes, devs, m, bandwidth):
    """Run time of every placement in devs [P][n]."""
    return np.array([runtime(n, src, dst, cost, nbytes, d, m, bandwidth) for d in devs])


def placements(n, src, dst, cost, nbytes, devs, m, bandwidth, mem_limit, scale):
    """Per placement in devs [P][n]: run time [P], peak memory per device [P][m],
    memory-penalised run time R(p) [P]."""
    out = [simulate(n, src, dst, cost, nbytes, d, m, bandwidth) for d in devs]
    r = np.array([o[0] for o in out])
    peaks = np.array([o[1] for o in out]).reshape(len(out), m)
    pen = np.array([penalised_runtime(a, float(pk.max()), mem_limit, scale) for a, pk in zip(r, peaks)])
    return r, peaks, pen
