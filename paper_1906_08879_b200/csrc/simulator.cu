// Run time of a placement under the event-based execution model of the Placeto
// paper's simulator (Appendix A.5): every device runs one operation at a time
// from a FIFO queue of runnable operations; every device's bus sends one output
// tensor at a time from a FIFO queue, overlapping with compute; an operation is
// runnable once all parents have finished and their outputs have arrived on its
// device; a transfer takes size / bandwidth; the result is the time stamp of the
// last Op-done event.
//
// One thread simulates one placement (the event loop is serial by nature; the
// batch of placements is the parallel dimension). At most one Op-done event per
// device and one Transfer-done event per bus are outstanding, so the event set is
// two arrays of m time stamps scanned for the earliest (equal stamps: the event
// created first). Queues are linked lists threaded through per-placement arrays
// in the workspace, which is interleaved by placement (element i of placement p
// at [i * P + p]) so that neighbouring threads touch neighbouring words. All
// times are doubles and are added and divided in the order the model states, so
// results are reproducible bit for bit.
//
// Readings where the paper is silent: one run time per operation; a tensor is
// sent once to each distinct device hosting a child; a free device or bus starts
// the head of its queue in the handler that filled it (a Wakeup with the current
// time stamp); operations without parents are queued in ascending id at time 0.
//
// Peak memory (Appendix A.5: the operations' start and end time stamps together
// with the tensor sizes predict the devices' peak memory; when a tensor is
// released is left open). Reading: a copy of an output tensor occupies the
// producer's device from the start of the producer until every child there has
// finished and every transfer of it is done; it occupies another device from
// the start of the transfer there until every child there has finished; outputs
// without children are never released. The memory-penalised run time of
// Appendix A.7 is R(p) = r if m <= M, r + c (m - M) otherwise, m the largest
// peak over the devices. Byte counts are doubles added and subtracted in event
// order (parents in ascending id inside an event): reproducible bit for bit.
#include <cfloat>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kThreads = 64;
constexpr int kMaxM = PLACETO_MAX_M;

// per placement: ints  pending[n], op_next[n], tr_op[T], tr_dst[T], tr_next[T], sent_mark[m * ?]
// with T = min(n_edges, n * (m - 1)) transfer records at most
__host__ __device__ inline size_t sim_ints(int n, int n_edges) {
    return 3 * (size_t)n + 3 * (size_t)n_edges;     // + tr_left[n]: transfers of a tensor not yet done
}

__global__ void __launch_bounds__(kThreads)
simulate_kernel(const SimArgs a) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= a.P) return;
    const int n = a.n, m = a.m, P = a.P;
    int *base = reinterpret_cast<int *>(a.workspace);
    auto at = [&](size_t i) -> int & { return base[i * P + p]; };
    const size_t o_pending = 0, o_next = n, o_trop = 2 * (size_t)n, o_trdst = o_trop + a.n_edges,
                 o_trnext = o_trdst + a.n_edges, o_trleft = o_trnext + a.n_edges;
    constexpr int kFinished = -1;            // value of pending[] once the operation has run
    const uint8_t *dev = a.dev + (size_t)p * n;

    // small per-device state in local memory
    int q_head[kMaxM], q_tail[kMaxM], t_head[kMaxM], t_tail[kMaxM];
    int run_op[kMaxM], run_tr[kMaxM];        // what the device / bus is busy with, -1 = free
    int op_seq[kMaxM], tr_seq[kMaxM];
    double op_end[kMaxM], tr_end[kMaxM];
    int sent[kMaxM];                          // last operation whose output was queued for the device
    double mem[kMaxM], peak[kMaxM];           // bytes held now / at most
    for (int d = 0; d < m; ++d) {
        q_head[d] = q_tail[d] = t_head[d] = t_tail[d] = -1;
        run_op[d] = run_tr[d] = -1;
        sent[d] = -1;
        mem[d] = peak[d] = 0.0;
    }
    auto hold = [&](int d, int o) {
        mem[d] += (double)a.bytes[o];
        if (mem[d] > peak[d]) peak[d] = mem[d];
    };
    // the copy of u's output on device d goes once no child there and no transfer needs it
    auto maybe_release = [&](int u, int d) {
        const int e0 = a.child_ptr[u], e1 = a.child_ptr[u + 1];
        if (e0 == e1) return;
        for (int e = e0; e < e1; ++e) {
            const int c = a.child[e];
            if (dev[c] == d && at(o_pending + c) != kFinished) return;
        }
        if (d == dev[u] && at(o_trleft + u) > 0) return;
        mem[d] -= (double)a.bytes[u];
    };
    int seq = 0, n_tr = 0, done = 0;
    double last = 0.0;

    auto push_op = [&](int d, int v) {
        at(o_next + v) = -1;
        if (q_tail[d] < 0) q_head[d] = v; else at(o_next + q_tail[d]) = v;
        q_tail[d] = v;
    };
    auto start_op = [&](int d, double now) {
        const int v = q_head[d];
        q_head[d] = at(o_next + v);
        if (q_head[d] < 0) q_tail[d] = -1;
        run_op[d] = v;
        hold(d, v);
        op_end[d] = now + (double)a.cost[v];
        op_seq[d] = seq++;
    };
    auto start_transfer = [&](int d, double now) {
        const int r = t_head[d];
        t_head[d] = at(o_trnext + r);
        if (t_head[d] < 0) t_tail[d] = -1;
        run_tr[d] = r;
        hold(at(o_trdst + r), at(o_trop + r));
        tr_end[d] = now + (double)a.bytes[at(o_trop + r)] / a.bandwidth;
        tr_seq[d] = seq++;
    };

    for (int v = 0; v < n; ++v) {
        at(o_pending + v) = a.n_parents[v];
        at(o_trleft + v) = 0;
        if (a.n_parents[v] == 0 && dev[v] < m) push_op(dev[v], v);
    }
    for (int d = 0; d < m; ++d)
        if (q_head[d] >= 0) start_op(d, 0.0);

    // every operation and every transfer is one event: the loop is bounded
    const long long max_events = (long long)n + a.n_edges + 1;
    for (long long it = 0; it < max_events; ++it) {
        // the earliest outstanding event; equal time stamps: the one created first
        int kind = -1, who = -1, best_seq = 0;
        double now = DBL_MAX;
        for (int d = 0; d < m; ++d) {
            if (run_op[d] >= 0 && (op_end[d] < now || (op_end[d] == now && op_seq[d] < best_seq))) {
                now = op_end[d]; kind = 0; who = d; best_seq = op_seq[d];
            }
            if (run_tr[d] >= 0 && (tr_end[d] < now || (tr_end[d] == now && tr_seq[d] < best_seq))) {
                now = tr_end[d]; kind = 1; who = d; best_seq = tr_seq[d];
            }
        }
        if (kind < 0) break;
        if (kind == 0) {                        // Op-done on device `who`
            const int d = who, o = run_op[d];
            run_op[d] = -1;
            ++done;
            last = now;
            at(o_pending + o) = kFinished;
            for (int e = a.parent_ptr[o]; e < a.parent_ptr[o + 1]; ++e)      // the inputs o read here
                if (dev[a.parent[e]] < m) maybe_release(a.parent[e], d);
            for (int e = a.child_ptr[o]; e < a.child_ptr[o + 1]; ++e) {
                const int c = a.child[e], dc = dev[c];
                if (dc >= m) continue;
                if (dc != d) {
                    if (sent[dc] != o && n_tr < a.n_edges) {   // the tensor goes to each device once
                        sent[dc] = o;
                        const int r = n_tr++;
                        at(o_trop + r) = o;
                        at(o_trdst + r) = dc;
                        at(o_trnext + r) = -1;
                        at(o_trleft + o) += 1;
                        if (t_tail[d] < 0) t_head[d] = r; else at(o_trnext + t_tail[d]) = r;
                        t_tail[d] = r;
                    }
                } else if (--at(o_pending + c) == 0) {
                    push_op(d, c);
                }
            }
            if (run_tr[d] < 0 && t_head[d] >= 0) start_transfer(d, now);
            if (q_head[d] >= 0) start_op(d, now);
        } else {                                // Transfer-done on the bus of device `who`
            const int d = who, r = run_tr[d];
            run_tr[d] = -1;
            const int o = at(o_trop + r), to = at(o_trdst + r);
            at(o_trleft + o) -= 1;
            maybe_release(o, d);
            for (int e = a.child_ptr[o]; e < a.child_ptr[o + 1]; ++e) {
                const int c = a.child[e];
                if (dev[c] == to && --at(o_pending + c) == 0) push_op(to, c);
            }
            if (run_op[to] < 0 && q_head[to] >= 0) start_op(to, now);
            if (t_head[d] >= 0) start_transfer(d, now);
        }
    }
    // a device id outside [0, m) leaves operations unplaced: report NaN
    const double nan = __longlong_as_double(0x7ff8000000000000LL);
    const bool ok = done == n;
    if (a.runtime) a.runtime[p] = ok ? last : nan;
    double top = 0.0;
    for (int d = 0; d < m; ++d) {
        if (a.peak_memory) a.peak_memory[(size_t)p * m + d] = ok ? peak[d] : nan;
        top = peak[d] > top ? peak[d] : top;
    }
    if (a.penalised) a.penalised[p] = !ok ? nan : (top <= a.mem_limit ? last : last + a.mem_scale * (top - a.mem_limit));
}

}  // namespace

size_t sim_workspace_bytes(int n, int n_edges, int m, int P) {
    (void)m;
    return std::max<size_t>(sim_ints(n, n_edges) * (size_t)P * sizeof(int), 256);
}

cudaError_t launch_simulator(const SimArgs &a, cudaStream_t stream) {
    simulate_kernel<<<(a.P + kThreads - 1) / kThreads, kThreads, 0, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace placeto
