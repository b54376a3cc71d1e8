// The "simple aggregator" policy of the paper's ablation (Sec. 4.3, "Alternative
// policy architectures", variant 1): a per-node network l over the raw
// features, summed over ALL nodes of the graph and squashed by h, then a head
// with softmax outputs:
//     a = h( sum_{u in V} l(x_u) ),  logits = head(a),  probs = softmax(logits).
// No message passing and no sets; the graph enters through its node count only.
//
// One block per state. The warps take the nodes round-robin (warp w: nodes w,
// w + W, ...), a lane owns output columns lane, lane + 32, ... of l and keeps
// their running sums in registers; the warps' sums are added in warp order, so
// the result is reproducible. l's weights sit in shared memory. h and the
// head are evaluated by the whole block through shared-memory vectors.
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kWarps = 8, kThreads = kWarps * 32;
constexpr int kMaxCols = (PLACETO_MAX_D + 31) / 32;

__device__ __forceinline__ float act_of(float v, int act) { return act == 0 ? fmaxf(v, 0.f) : v; }

// y[0 .. out) = W^T x + b over the whole block (x, y in shared memory), optional activation
__device__ void block_dense(const float *W, const float *b, int in, int out, const float *x, float *y, int act,
                            bool apply) {
    for (int j = threadIdx.x; j < out; j += blockDim.x) {
        float s = b[j];
        for (int k = 0; k < in; ++k) s = fmaf(x[k], W[(size_t)k * out + j], s);
        y[j] = apply ? act_of(s, act) : s;
    }
    __syncthreads();
}

// One or two layers (Appendix A.7 convention of the library); result in `y`, `tmp` holds the hidden layer.
__device__ void block_mlp(const DevMlp &m, const float *x, float *tmp, float *y) {
    if (m.n_layers == 2) {
        block_dense(m.W1, m.b1, m.in_dim, m.hidden_dim, x, tmp, m.act, true);
        block_dense(m.W2, m.b2, m.hidden_dim, m.out_dim, tmp, y, m.act, m.final_act != 0);
    } else {
        block_dense(m.W1, m.b1, m.in_dim, m.out_dim, x, y, m.act, m.final_act != 0);
    }
}

struct AggArgs {
    DevMlp l, h, head;
    const float *X;
    float *logits, *probs;
    int n, B, F, d, m;
    int l_in_smem;      // l staged in shared memory
    int vec_floats;     // floats of one shared-memory vector (the widest layer)
};

__global__ void __launch_bounds__(kThreads) simple_aggregator_kernel(const AggArgs a) {
    extern __shared__ __align__(16) float smem[];
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int F = a.F, d = a.d;
    // shared memory: [l's networks][per-warp input row + hidden row][warp sums][three block vectors]
    float *w = smem;
    const float *W1 = a.l.W1, *b1 = a.l.b1, *W2 = a.l.W2, *b2 = a.l.b2;
    const int lh = a.l.n_layers == 2 ? a.l.hidden_dim : d;
    if (a.l_in_smem) {
        auto stage = [&](const float *src, size_t count) {
            float *dst = w;
            for (size_t k = threadIdx.x; k < count; k += blockDim.x) dst[k] = src[k];
            w += (count + 3) & ~size_t(3);
            return (const float *)dst;
        };
        W1 = stage(a.l.W1, (size_t)F * lh);
        b1 = stage(a.l.b1, lh);
        if (a.l.n_layers == 2) {
            W2 = stage(a.l.W2, (size_t)lh * d);
            b2 = stage(a.l.b2, d);
        }
    }
    const int row_floats = ((F + 3) & ~3) + ((lh + 3) & ~3);
    float *row = w + (size_t)warp * row_floats, *hid = row + ((F + 3) & ~3);
    float *sums = w + (size_t)kWarps * row_floats;            // [kWarps][d]
    float *v0 = sums + (size_t)kWarps * ((d + 3) & ~3), *v1 = v0 + a.vec_floats, *v2 = v1 + a.vec_floats;
    __syncthreads();

    float acc[kMaxCols];
#pragma unroll
    for (int t = 0; t < kMaxCols; ++t) acc[t] = 0.f;
    for (int u = warp; u < a.n; u += kWarps) {
        const float *x = a.X + ((size_t)u * a.B + b) * F;
        for (int k = lane; k < F; k += 32) row[k] = x[k];
        __syncwarp();
        const float *in = row;
        int in_dim = F;
        const float *W = W1, *bias = b1;
        if (a.l.n_layers == 2) {
            for (int j = lane; j < lh; j += 32) {
                float s = bias[j];
                for (int k = 0; k < F; ++k) s = fmaf(in[k], W[k * lh + j], s);
                hid[j] = act_of(s, a.l.act);
            }
            __syncwarp();
            in = hid; in_dim = lh; W = W2; bias = b2;
        }
#pragma unroll
        for (int t = 0; t < kMaxCols; ++t) {
            const int j = lane + 32 * t;
            if (j < d) {
                float s = bias[j];
                for (int k = 0; k < in_dim; ++k) s = fmaf(in[k], W[k * d + j], s);
                acc[t] += a.l.final_act ? act_of(s, a.l.act) : s;
            }
        }
        __syncwarp();
    }
#pragma unroll
    for (int t = 0; t < kMaxCols; ++t) {
        const int j = lane + 32 * t;
        if (j < d) sums[warp * ((d + 3) & ~3) + j] = acc[t];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        float s = 0.f;
        for (int wv = 0; wv < kWarps; ++wv) s += sums[wv * ((d + 3) & ~3) + j];   // warp order: reproducible
        v0[j] = s;
    }
    __syncthreads();
    block_mlp(a.h, v0, v1, v2);          // a = h(sum)
    block_mlp(a.head, v2, v1, v0);       // logits
    if (threadIdx.x == 0) {
        float mx = v0[0];
        for (int k = 1; k < a.m; ++k) mx = fmaxf(mx, v0[k]);
        float tot = 0.f;
        for (int k = 0; k < a.m; ++k) tot += expf(v0[k] - mx);
        for (int k = 0; k < a.m; ++k) {
            a.logits[(size_t)b * a.m + k] = v0[k];
            if (a.probs) a.probs[(size_t)b * a.m + k] = expf(v0[k] - mx) / tot;
        }
    }
}

}  // namespace

cudaError_t launch_simple_aggregator(const DevMlp &l, const DevMlp &h, const DevMlp &head, const float *X, int n,
                                     int B, int F, int d, int m, float *logits, float *probs, const DeviceInfo &di,
                                     cudaStream_t stream) {
    AggArgs a;
    a.l = l; a.h = h; a.head = head;
    a.X = X; a.logits = logits; a.probs = probs;
    a.n = n; a.B = B; a.F = F; a.d = d; a.m = m;
    const int lh = l.n_layers == 2 ? l.hidden_dim : d;
    int widest = std::max(d, m);
    for (const DevMlp *net : {&h, &head}) widest = std::max(widest, net->n_layers == 2 ? net->hidden_dim : net->out_dim);
    a.vec_floats = (widest + 3) & ~3;
    const size_t row_floats = ((F + 3) & ~3) + ((lh + 3) & ~3);
    const size_t fixed = kWarps * row_floats + (size_t)kWarps * ((d + 3) & ~3) + 3 * (size_t)a.vec_floats;
    const size_t l_floats = ((mlp_floats(l) + 15) & ~size_t(15));
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    a.l_in_smem = (fixed + l_floats) * sizeof(float) <= budget;
    const size_t smem = (fixed + (a.l_in_smem ? l_floats : 0)) * sizeof(float);
    if (smem > budget) return cudaErrorNotSupported;
    cudaError_t err = cudaFuncSetAttribute(simple_aggregator_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    simple_aggregator_kernel<<<B, kThreads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace placeto
