// The MDP transition of a placement episode (Sec. 2.1 of the Placeto paper) on
// the device: after the policy kernels have produced the logits of step t, one
// thread per episode picks the current node's device (argmax, or an inverse-CDF
// sample driven by a caller-supplied uniform number), writes it into the
// placement, marks the node visited, records the log-probability of the choice
// and makes the next node of the visiting order current. With it a whole episode
// runs as a stream of launches without a host round trip per step.
//
// Two forms. Where the step's kernels take compact states (the d = 32 sweep and pooling
// kernels with the fast head kernel), there is no feature tensor at all: the state of the
// E episodes is one byte per (node, episode) plus the current node, the kernels build the
// features on the fly, and the transition itself is the head kernel's last step (see
// EpisodeStep); this file then only converts the placement to and from compact states.
// Elsewhere the transition is the kernel below: a step changes the raw features of two
// nodes only (the node just placed: device one-hot, current flag off, visited flag on; the
// next node: current flag on), so the thread of an episode patches those rows of X in
// place and the feature tensor is built once per episode, not once per step.
#include <cmath>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kThreads = 128;

// placed[e][:] = 0 and cur[e] = order[0] for every episode
__global__ void episode_begin_kernel(int n, int E, const int *__restrict__ order,
                                     uint8_t *__restrict__ placed, int *__restrict__ cur) {
    const size_t total = (size_t)E * n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x)
        placed[i] = 0;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < E) cur[e] = order[0];
}

// Greedy: the largest logit, the lowest index among equals. Sampling: with
// p = softmax(logits) (max-subtracted, FP32, summed in index order), the first
// index k with p_0 + .. + p_k > u, the last index if rounding leaves none.
__global__ void episode_step_kernel(EpisodeArgs a, int t) {
    dependents_may_start();
    dependency_wait();          // the logits come from a kernel that may still be running
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= a.E) return;
    const int m = a.m, n = a.n;
    const float *l = a.logits + (size_t)e * m;
    const int v = a.order[t];
    float mx = l[0];
    int best = 0;
    for (int k = 1; k < m; ++k)
        if (l[k] > mx) { mx = l[k]; best = k; }
    float tot = 0.f;
    for (int k = 0; k < m; ++k) tot += expf(l[k] - mx);
    int action = best;
    if (a.uniforms != nullptr) {
        const float u = a.uniforms[(size_t)e * n + t];
        float cum = 0.f;
        action = m - 1;
        for (int k = 0; k < m; ++k) {
            cum += expf(l[k] - mx) / tot;
            if (cum > u) { action = k; break; }
        }
    }
    if (a.logp != nullptr) a.logp[(size_t)e * n + t] = (l[action] - mx) - logf(tot);
    if (a.actions != nullptr) a.actions[(size_t)e * n + t] = (uint8_t)action;
    const int F = m + 4;        // x = [cost, bytes, one-hot(m), is-current, is-visited]
    if (v >= 0 && v < n) {      // an id outside the graph leaves the placement alone
        a.dev[(size_t)e * n + v] = (uint8_t)action;
        a.placed[(size_t)e * n + v] = 1;
        float *x = a.X + ((size_t)v * a.E + e) * F;
        for (int k = 0; k < m; ++k) x[2 + k] = k == action ? 1.f : 0.f;
        x[2 + m] = 0.f;
        x[3 + m] = 1.f;
    }
    if (t + 1 < n) {
        const int next = a.order[t + 1];
        a.cur[e] = next;
        if (next >= 0 && next < n) a.X[((size_t)next * a.E + e) * F + 2 + m] = 1.f;
    }
}

// compact states from the initial placement: state[v][e] = device (63 for an id that no device
// carries: its one-hot is all zero), nothing visited; cur[e] = order[0]
__global__ void episode_begin_compact_kernel(int n, int E, const int *__restrict__ order,
                                             const uint8_t *__restrict__ dev, uint8_t *__restrict__ state,
                                             int *__restrict__ cur) {
    const size_t total = (size_t)E * n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t v = i / E, e = i - v * E;
        const uint8_t d = dev[e * n + v];
        state[i] = d < 63 ? d : 63;
    }
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < E) cur[e] = order[0];
}

__global__ void episode_end_compact_kernel(int n, int E, const uint8_t *__restrict__ state,
                                           uint8_t *__restrict__ dev) {
    dependency_wait();
    const size_t total = (size_t)E * n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t e = i / n, v = i - e * n;
        // a node that was never visited keeps the device it came with (63 stood for any id >= 63)
        const uint8_t s = state[v * E + e];
        if (s & 0x80) dev[i] = s & 63;
    }
}

}  // namespace

cudaError_t launch_episode_begin_compact(int n, int E, const int *order, const uint8_t *dev, uint8_t *state,
                                         int *cur, cudaStream_t stream) {
    const int blocks = std::max(1, std::min(2048, (int)(((size_t)E * n + kThreads - 1) / kThreads)));
    const int need = (E + kThreads - 1) / kThreads;       // every episode needs its thread
    episode_begin_compact_kernel<<<std::max(blocks, need), kThreads, 0, stream>>>(n, E, order, dev, state, cur);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_episode_end_compact(int n, int E, const uint8_t *state, uint8_t *dev, cudaStream_t stream) {
    const int blocks = std::max(1, std::min(2048, (int)(((size_t)E * n + kThreads - 1) / kThreads)));
    cudaError_t err = launch_overlapped(true, episode_end_compact_kernel, dim3(blocks), dim3(kThreads), 0, stream,
                                        n, E, state, dev);
    count_launch();
    return err;
}

cudaError_t launch_episode_begin(const EpisodeArgs &a, cudaStream_t stream) {
    const int blocks = std::max(1, std::min(1024, (int)(((size_t)a.E * a.n + kThreads - 1) / kThreads)));
    const int need = (a.E + kThreads - 1) / kThreads;       // every episode needs its thread
    episode_begin_kernel<<<std::max(blocks, need), kThreads, 0, stream>>>(a.n, a.E, a.order, a.placed, a.cur);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_episode_step(const EpisodeArgs &a, int t, cudaStream_t stream) {
    // always preceded by this library's head kernel on the same stream
    cudaError_t err = launch_overlapped(true, episode_step_kernel, dim3((a.E + kThreads - 1) / kThreads),
                                        dim3(kThreads), 0, stream, a, t);
    count_launch();
    return err;
}

}  // namespace placeto
