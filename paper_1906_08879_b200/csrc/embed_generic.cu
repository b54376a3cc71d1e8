// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper), for any widths:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]),
// top-down (nbr = parents) and bottom-up (nbr = children) with separate
// parameters. What a node sends depends on the node only, so the message m_u is
// computed once per node and state and kept in the workspace; a node's row is
// then gather-sum -> g -> store h -> f -> store m.
//
// States never interact, so the batch is cut into slices: a block owns one
// direction and one slice of states. Three schedules share the row code:
//   PER_LEVEL    one launch per level (the level order comes from the launches)
//   SLICED       one persistent launch; a block walks every level of its
//                direction, ordering them with __syncthreads() only
//   COOPERATIVE  one persistent cooperative launch; the nodes of a level are also
//                spread over several blocks, with a grid-wide sync per level
// This file is the dimension-generic fallback: one thread per output element,
// weights staged in shared memory when they fit.
#include <cooperative_groups.h>

#include <algorithm>

#include "kernels.cuh"

namespace cg = cooperative_groups;

namespace placeto {

namespace {

constexpr int kThreads = 256;

struct GenericPlan {
    int S;            // states per slice
    int n_slices;
    int node_splits;  // blocks sharing a level (cooperative), else 1
    int rows_cap;     // rows (node, state) per pass through the buffers
    int width;        // floats per buffered row
    int weights_in_smem;
    int level_begin, level_end;
    // Synchronous rounds (all nodes at once from the previous round's messages):
    // 0 off; 1 a round: h = g(sum of M_in), M_out = f([h || x]); 2 the start:
    // h = 0 (not stored), M_out = f([0 || x]).
    int round_mode;
    const float *M_in[2];
    float *M_out[2];
    size_t smem_bytes;
};

// dst[r][0..out) = act(bias + src[r][0..in) W), W[in][out]; one thread per element.
__device__ __forceinline__ void dense(const float *W, const float *bias, int in, int out,
                                      bool relu, const float *src, float *dst, int stride,
                                      int rows) {
    for (int idx = threadIdx.x; idx < rows * out; idx += blockDim.x) {
        const int r = idx / out, j = idx - r * out;
        const float *v = src + r * stride;
        float acc = bias[j];
        for (int k = 0; k < in; ++k) acc = fmaf(v[k], W[k * out + j], acc);
        dst[r * stride + j] = relu ? fmaxf(acc, 0.f) : acc;
    }
}

// Applies a network to `rows` buffered rows; returns the buffer holding the result.
__device__ __forceinline__ float *apply_mlp(const DevMlp &net, const float *W1, const float *b1,
                                            const float *W2, const float *b2, float *cur,
                                            float *nxt, int stride, int rows) {
    const bool relu = net.act == 0;
    const bool act1 = relu && (net.n_layers == 2 || net.final_act);
    dense(W1, b1, net.in_dim, net.hidden_dim, act1, cur, nxt, stride, rows);
    __syncthreads();
    if (net.n_layers == 1) return nxt;
    dense(W2, b2, net.hidden_dim, net.out_dim, relu && net.final_act, nxt, cur, stride, rows);
    __syncthreads();
    return cur;
}

template <bool kCooperative>
__global__ void __launch_bounds__(kThreads)
embed_generic_kernel(const EmbedArgs a, const GenericPlan p) {
    extern __shared__ __align__(16) float smem[];
    const int dir = blockIdx.y;
    const int slice = blockIdx.x / p.node_splits;
    const int split = blockIdx.x - slice * p.node_splits;
    const int b0 = slice * p.S;
    const int nb = min(p.S, a.B - b0);
    const DevLevels lv = a.lv[dir];
    const DevMlp f = a.f[dir], g = a.g[dir];
    const int d = a.d, F = a.F, B = a.B;
    const float *__restrict__ X = a.X;
    float *__restrict__ H = a.H[dir];
    const float *Min = p.round_mode ? p.M_in[dir] : a.M[dir];
    float *M = p.round_mode ? p.M_out[dir] : a.M[dir];

    // Stage the direction's weights once per block.
    const float *fW1 = f.W1, *fb1 = f.b1, *fW2 = f.W2, *fb2 = f.b2;
    const float *gW1 = g.W1, *gb1 = g.b1, *gW2 = g.W2, *gb2 = g.b2;
    float *buf = smem;
    if (p.weights_in_smem) {
        float *w = smem;
        auto stage = [&](const float *src, size_t count) {
            float *dst = w;
            for (size_t i = threadIdx.x; i < count; i += blockDim.x) dst[i] = src[i];
            w += (count + 3) & ~size_t(3);
            return dst;
        };
        fW1 = stage(f.W1, (size_t)f.in_dim * f.hidden_dim);
        fb1 = stage(f.b1, f.hidden_dim);
        if (f.n_layers == 2) { fW2 = stage(f.W2, (size_t)f.hidden_dim * f.out_dim); fb2 = stage(f.b2, f.out_dim); }
        gW1 = stage(g.W1, (size_t)g.in_dim * g.hidden_dim);
        gb1 = stage(g.b1, g.hidden_dim);
        if (g.n_layers == 2) { gW2 = stage(g.W2, (size_t)g.hidden_dim * g.out_dim); gb2 = stage(g.b2, g.out_dim); }
        buf = w;
    }
    float *bufA = buf, *bufB = buf + (size_t)p.rows_cap * p.width;
    const int stride = p.width;
    __syncthreads();

    // In the cooperative schedule every block runs the same number of rounds.
    const int last = kCooperative ? p.level_end : min(p.level_end, lv.n_levels);
    for (int level = p.level_begin; level < last; ++level) {
        if (level < lv.n_levels) {
            // a synchronous round treats all nodes as one level
            const int p0 = p.round_mode ? 0 : lv.level_ptr[level];
            const int p1 = p.round_mode ? a.n : lv.level_ptr[level + 1];
            const int width_l = p1 - p0;
            const int mine = (width_l - split + p.node_splits - 1) / p.node_splits;  // nodes p0+split+q*splits
            const int rows_total = mine > 0 ? mine * nb : 0;
            for (int r0 = 0; r0 < rows_total; r0 += p.rows_cap) {
                const int rows = min(p.rows_cap, rows_total - r0);
                // gather: s = sum of the neighbours' messages
                for (int idx = threadIdx.x; idx < rows * d; idx += blockDim.x) {
                    const int r = idx / d, j = idx - r * d;
                    const int q = (r0 + r) / nb, b = b0 + (r0 + r) - q * nb;
                    const int pos = p0 + split + q * p.node_splits;
                    float s = 0.f;
                    if (p.round_mode != 2)
                        for (int e = lv.nbr_ptr[pos]; e < lv.nbr_ptr[pos + 1]; ++e)
                            s += __ldcg(Min + ((size_t)lv.nbr[e] * B + b) * d + j);
                    bufA[r * stride + j] = s;
                }
                __syncthreads();
                float *h = p.round_mode == 2 ? bufA
                                             : apply_mlp(g, gW1, gb1, gW2, gb2, bufA, bufB, stride, rows);
                float *other = (h == bufA) ? bufB : bufA;
                // store h and append the node's raw features: [h || x]
                for (int idx = threadIdx.x; idx < rows * (d + F); idx += blockDim.x) {
                    const int r = idx / (d + F), j = idx - r * (d + F);
                    const int q = (r0 + r) / nb, b = b0 + (r0 + r) - q * nb;
                    const int v = lv.order[p0 + split + q * p.node_splits];
                    if (j < d) { if (p.round_mode != 2) H[((size_t)v * B + b) * d + j] = h[r * stride + j]; }
                    else h[r * stride + j] = X[((size_t)v * B + b) * F + (j - d)];
                }
                __syncthreads();
                const float *msg = apply_mlp(f, fW1, fb1, fW2, fb2, h, other, stride, rows);
                for (int idx = threadIdx.x; idx < rows * d; idx += blockDim.x) {
                    const int r = idx / d, j = idx - r * d;
                    const int q = (r0 + r) / nb, b = b0 + (r0 + r) - q * nb;
                    const int v = lv.order[p0 + split + q * p.node_splits];
                    M[((size_t)v * B + b) * d + j] = msg[r * stride + j];
                }
                __syncthreads();
            }
        }
        if (kCooperative) cg::this_grid().sync();
    }
}

int slices_for(int B, int target) { return std::max(1, std::min(B, target)); }

}  // namespace

namespace {

// Row buffers, weight staging and state slices common to every schedule.
GenericPlan base_plan(const EmbedArgs &a, const DeviceInfo &di) {
    GenericPlan p;
    const int max_hidden = std::max(std::max(a.f[0].hidden_dim, a.f[1].hidden_dim),
                                    std::max(a.g[0].hidden_dim, a.g[1].hidden_dim));
    p.width = (std::max(a.d + a.F, max_hidden) + 3) & ~3;
    size_t wfloats = 0;
    for (int dir = 0; dir < 2; ++dir) {
        size_t s = 0;
        for (const DevMlp *m : {&a.f[dir], &a.g[dir]}) {
            s += (((size_t)m->in_dim * m->hidden_dim + 3) & ~size_t(3)) + ((m->hidden_dim + 3) & ~3);
            if (m->n_layers == 2)
                s += (((size_t)m->hidden_dim * m->out_dim + 3) & ~size_t(3)) + ((m->out_dim + 3) & ~3);
        }
        wfloats = std::max(wfloats, s);
    }
    const size_t budget = (size_t)std::min(di.max_smem_optin, 200 * 1024);
    p.rows_cap = 32;
    size_t buf_bytes = 2ull * p.rows_cap * p.width * sizeof(float);
    p.weights_in_smem = (wfloats * sizeof(float) + buf_bytes <= budget) ? 1 : 0;
    p.smem_bytes = buf_bytes + (p.weights_in_smem ? wfloats * sizeof(float) : 0);

    const int target = std::max(1, di.sm_count / 2);   // blocks per direction
    const int n_slices = slices_for(a.B, target);
    p.S = (a.B + n_slices - 1) / n_slices;
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.node_splits = 1;
    p.round_mode = 0;
    p.M_in[0] = p.M_in[1] = nullptr;
    p.M_out[0] = p.M_out[1] = nullptr;
    return p;
}

}  // namespace

cudaError_t launch_embed_generic(const EmbedArgs &a, const DeviceInfo &di, unsigned schedule,
                                 cudaStream_t stream) {
    GenericPlan p = base_plan(a, di);
    const int max_levels = std::max(a.lv[0].n_levels, a.lv[1].n_levels);

    cudaError_t err;
    if (schedule == PLACETO_COOPERATIVE) {
        auto kern = embed_generic_kernel<true>;
        err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
        if (err != cudaSuccess) return err;
        int per_sm = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, p.smem_bytes);
        if (err != cudaSuccess) return err;
        const int capacity = per_sm * di.sm_count;
        if (capacity < 2 * p.n_slices) {
            // too many slices to be co-resident: widen the slices
            const int s2 = std::max(1, capacity / 2);
            p.S = (a.B + s2 - 1) / s2;
            p.n_slices = (a.B + p.S - 1) / p.S;
        }
        if (capacity < 2 * p.n_slices || capacity < 2) return cudaErrorCooperativeLaunchTooLarge;
        p.node_splits = std::max(1, capacity / (2 * p.n_slices));
        p.level_begin = 0;
        p.level_end = max_levels;
        dim3 grid(p.n_slices * p.node_splits, 2);
        void *params[] = {(void *)&a, (void *)&p};
        err = cudaLaunchCooperativeKernel((void *)kern, grid, dim3(kThreads), params, p.smem_bytes, stream);
        count_launch();
        return err;
    }
    auto kern = embed_generic_kernel<false>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    dim3 grid(p.n_slices, 2);
    if (schedule == PLACETO_PER_LEVEL) {
        for (int level = 0; level < max_levels; ++level) {
            p.level_begin = level;
            p.level_end = level + 1;
            embed_generic_kernel<false><<<grid, kThreads, p.smem_bytes, stream>>>(a, p);
            count_launch();
        }
        return cudaGetLastError();
    }
    p.level_begin = 0;
    p.level_end = max_levels;
    embed_generic_kernel<false><<<grid, kThreads, p.smem_bytes, stream>>>(a, p);
    count_launch();
    return cudaGetLastError();
}

// The synchronous form of step 2 (Sec. 2.2 step 2: the updates are repeated k
// times): H^0 = 0 and H^r_v = g(sum_u f([H^(r-1)_u || x_u])) for every node at
// once. One launch per round over all (node, state) rows, the nodes of a state
// slice spread over several blocks; messages alternate between two buffers per
// direction (msg[2 * dir], msg[2 * dir + 1]).
cudaError_t launch_embed_rounds(const EmbedArgs &a, const DeviceInfo &di, int rounds, float *const msg[4],
                                cudaStream_t stream) {
    if (embed_d32_applicable(a)) {
        const cudaError_t e = launch_embed_rounds_d32(a, di, rounds, msg, stream);
        if (e != cudaErrorNotSupported) return e;
    }
    GenericPlan p = base_plan(a, di);
    // enough blocks per direction to fill the device about four times over
    p.node_splits = std::max(1, std::min(a.n, (4 * di.sm_count + p.n_slices - 1) / p.n_slices));
    p.level_begin = 0;
    p.level_end = 1;
    auto kern = embed_generic_kernel<false>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    dim3 grid(p.n_slices * p.node_splits, 2);
    for (int r = 0; r <= rounds; ++r) {
        p.round_mode = r == 0 ? 2 : 1;
        for (int dir = 0; dir < 2; ++dir) {
            p.M_in[dir] = msg[2 * dir + ((r + 1) & 1)];
            p.M_out[dir] = msg[2 * dir + (r & 1)];
        }
        kern<<<grid, kThreads, p.smem_bytes, stream>>>(a, p);
        count_launch();
        err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

}  // namespace placeto
