// Step 3 and the head of the policy (Sec. 2.2 step 3 and Appendix A.7 of the
// Placeto paper), for any widths.
//
// With e_u = [h_down_u || h_up_u || x_u] and c the state's current node,
//   a_i = h_i( sum_{u in S_i(c)} l_i(e_u) ),  i = can-reach-c / reachable-from-c / neither,
//   logits = head([e_c || a_0 || a_1 || a_2]),  probs = softmax(logits).
// Kernel 1 cuts the nodes into chunks and writes, per chunk and state, the three
// partial sums of l_i(e_u) (one warp per state, lanes over the output columns,
// the set of each node read from the relation row of c). Kernel 2 adds the
// chunks in a fixed order (deterministic, no atomics), applies h_i, the head and
// the softmax, eight states per block so that each weight is read once per block.
#include <cuda_pipeline.h>

#include <algorithm>
#include <cmath>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kPoolThreads = 256;
constexpr int kPoolWarps = kPoolThreads / 32;
constexpr int kMaxCols = PLACETO_MAX_D / 32;   // output columns per lane
constexpr int kHeadThreads = 512;
constexpr int kHeadStates = 8;      // states finished per block of the head kernel

struct PoolPlan {
    int states_per_block;
    int weights_in_smem;
    int e_stride;       // floats of the per-warp row buffer (input row + hidden row)
    size_t smem_bytes;
};

__global__ void __launch_bounds__(kPoolThreads)
pool_partial_kernel(const PoolArgs a, const PoolPlan p) {
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    const int d = a.d, F = a.F, n = a.n, B = a.B;
    const int E = 2 * d + F;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // l_i weights: staged contiguously per set when they fit
    const float *W1[3], *b1[3], *W2[3], *b2[3];
    float *w = smem;
    for (int i = 0; i < 3; ++i) {
        W1[i] = a.l[i].W1; b1[i] = a.l[i].b1; W2[i] = a.l[i].W2; b2[i] = a.l[i].b2;
        if (p.weights_in_smem) {
            auto stage = [&](const float *src, size_t count) {
                float *dst = w;
                for (size_t k = threadIdx.x; k < count; k += blockDim.x) dst[k] = src[k];
                w += (count + 3) & ~size_t(3);
                return (const float *)dst;
            };
            W1[i] = stage(a.l[i].W1, (size_t)a.l[i].in_dim * a.l[i].hidden_dim);
            b1[i] = stage(a.l[i].b1, a.l[i].hidden_dim);
            if (a.l[i].n_layers == 2) {
                W2[i] = stage(a.l[i].W2, (size_t)a.l[i].hidden_dim * a.l[i].out_dim);
                b2[i] = stage(a.l[i].b2, a.l[i].out_dim);
            }
        }
    }
    float *row = w + (size_t)warp * p.e_stride;   // [E] input row, then hidden row
    float *hid = row + ((E + 3) & ~3);
    __syncthreads();

    const int chunk = blockIdx.x;
    const int u0 = chunk * a.chunk_nodes, u1 = min(n, u0 + a.chunk_nodes);
    const int bs0 = blockIdx.y * p.states_per_block;
    const int bs1 = min(B, bs0 + p.states_per_block);
    for (int b = bs0 + warp; b < bs1; b += kPoolWarps) {
        const int c = a.cur[b];
        float acc[3][kMaxCols];
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int t = 0; t < kMaxCols; ++t) acc[i][t] = 0.f;
        const bool valid = c >= 0 && c < n;
        if (valid) {
            const uint8_t *rel = a.relation + (size_t)c * n;
            for (int u = u0; u < u1; ++u) {
                const int i = rel[u];
                if (i == 3) continue;
                const float *hd = a.H[0] + ((size_t)u * B + b) * d;
                const float *hu = a.H[1] + ((size_t)u * B + b) * d;
                const float *x = a.X + ((size_t)u * B + b) * F;
                for (int k = lane; k < d; k += 32) { row[k] = hd[k]; row[d + k] = hu[k]; }
                for (int k = lane; k < F; k += 32) row[2 * d + k] = x[k];
                __syncwarp();
                const DevMlp &net = a.l[i];
                const bool relu = net.act == 0;
                const float *in = row;
                int in_dim = E;
                const float *W = W1[i], *bias = b1[i];
                if (net.n_layers == 2) {
                    for (int j = lane; j < net.hidden_dim; j += 32) {
                        float s = bias[j];
                        for (int k = 0; k < E; ++k) s = fmaf(in[k], W[k * net.hidden_dim + j], s);
                        hid[j] = relu ? fmaxf(s, 0.f) : s;
                    }
                    __syncwarp();
                    in = hid; in_dim = net.hidden_dim; W = W2[i]; bias = b2[i];
                }
#pragma unroll
                for (int t = 0; t < kMaxCols; ++t) {
                    const int j = lane + 32 * t;
                    if (j < d) {
                        float s = bias[j];
                        for (int k = 0; k < in_dim; ++k) s = fmaf(in[k], W[k * d + j], s);
                        if (relu && net.final_act) s = fmaxf(s, 0.f);
#pragma unroll
                        for (int ii = 0; ii < 3; ++ii) acc[ii][t] += (ii == i) ? s : 0.f;
                    }
                }
                __syncwarp();
            }
        }
        float *out = a.partial + ((size_t)chunk * B + b) * 3 * d;
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int t = 0; t < kMaxCols; ++t) {
                const int j = lane + 32 * t;
                if (j < d) out[i * d + j] = valid ? acc[i][t] : nanf("");
            }
    }
}

// dst[s][0..out) = act(bias + src[s][0..in) W) for the kHeadStates rows of a block.
// Wide layers: a thread owns one output column and one part of the inner
// dimension for all rows, so each weight is read once per block (coalesced over
// columns) with eight loads in flight; the parts are then added in a fixed order
// through `red`. Narrow layers (the device logits): one warp per (row, column),
// the lanes split the inner dimension and combine with a shuffle reduction.
// Not inlined on purpose: the kernel calls it eight times and runs each call once,
// so one shared copy of the code keeps the instruction fetches (cold after an L2
// flush) to a single pass.
__device__ __noinline__ void head_dense(const float *__restrict__ W,
                                           const float *__restrict__ bias, int in, int out,
                                           bool relu, const float *src, int src_stride, float *dst,
                                           int dst_stride, float *red) {
    if (out >= 32) {
        // parts * out <= blockDim.x, so `red` (blockDim.x * kHeadStates floats) holds
        // every partial product; layers wider than the block take several column passes
        const int parts = max(1, min((int)blockDim.x / out, (in + 7) / 8));
        const int per = ((in + parts - 1) / parts + 3) & ~3;
        const bool vec = (reinterpret_cast<uintptr_t>(src) & 15) == 0 && (src_stride & 3) == 0;
        for (int j0 = 0; j0 < out; j0 += blockDim.x) {
            const int cols = min(out - j0, (int)blockDim.x);
            const int part = threadIdx.x / cols, jl = threadIdx.x - part * cols;
            const int j = j0 + jl;
            if (part < parts) {
                float acc[kHeadStates];
#pragma unroll
                for (int s = 0; s < kHeadStates; ++s) acc[s] = 0.f;
                const int k1 = min(in, (part + 1) * per);
                int k = part * per;
                for (; k + 8 <= k1; k += 8) {
                    float wv[8];
#pragma unroll
                    for (int t = 0; t < 8; ++t) wv[t] = W[(size_t)(k + t) * out + j];
#pragma unroll
                    for (int s = 0; s < kHeadStates; ++s) {
                        const float *v = src + s * src_stride + k;
                        float4 v0, v1;
                        if (vec) {
                            v0 = *reinterpret_cast<const float4 *>(v);
                            v1 = *reinterpret_cast<const float4 *>(v + 4);
                        } else {
                            v0 = make_float4(v[0], v[1], v[2], v[3]);
                            v1 = make_float4(v[4], v[5], v[6], v[7]);
                        }
                        acc[s] = fmaf(v0.x, wv[0], acc[s]); acc[s] = fmaf(v0.y, wv[1], acc[s]);
                        acc[s] = fmaf(v0.z, wv[2], acc[s]); acc[s] = fmaf(v0.w, wv[3], acc[s]);
                        acc[s] = fmaf(v1.x, wv[4], acc[s]); acc[s] = fmaf(v1.y, wv[5], acc[s]);
                        acc[s] = fmaf(v1.z, wv[6], acc[s]); acc[s] = fmaf(v1.w, wv[7], acc[s]);
                    }
                }
                for (; k < k1; ++k) {
                    const float w0 = W[(size_t)k * out + j];
#pragma unroll
                    for (int s = 0; s < kHeadStates; ++s)
                        acc[s] = fmaf(src[s * src_stride + k], w0, acc[s]);
                }
#pragma unroll
                for (int s = 0; s < kHeadStates; ++s)
                    red[(part * kHeadStates + s) * cols + jl] = acc[s];
            }
            __syncthreads();
            for (int i = threadIdx.x; i < kHeadStates * cols; i += blockDim.x) {
                const int s = i / cols, jj = i - s * cols;
                float acc = bias[j0 + jj];
                for (int q = 0; q < parts; ++q) acc += red[(q * kHeadStates + s) * cols + jj];
                dst[s * dst_stride + j0 + jj] = relu ? fmaxf(acc, 0.f) : acc;
            }
            __syncthreads();
        }
    } else {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
        for (int item = warp; item < out * kHeadStates; item += nw) {
            const int s = item / out, j = item - s * out;
            float acc = 0.f;
            for (int k = lane; k < in; k += 32)
                acc = fmaf(src[s * src_stride + k], W[(size_t)k * out + j], acc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            acc += bias[j];
            if (lane == 0) dst[s * dst_stride + j] = relu ? fmaxf(acc, 0.f) : acc;
        }
    }
    __syncthreads();
}

// Asks for `count` floats to be brought into L2 (the block's threads share the lines).
__device__ __forceinline__ void prefetch_l2(const float *p, size_t count) {
    const char *base = reinterpret_cast<const char *>(p);
    for (size_t off = (size_t)threadIdx.x * 128; off < count * sizeof(float); off += (size_t)blockDim.x * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
}

__device__ __forceinline__ void head_mlp(const DevMlp &net, const float *in, int in_stride,
                                         float *tmp, int tmp_stride, float *out, int out_stride,
                                         float *red) {
    const bool relu = net.act == 0;
    if (net.n_layers == 1) {
        head_dense(net.W1, net.b1, net.in_dim, net.out_dim, relu && net.final_act, in, in_stride,
                   out, out_stride, red);
        return;
    }
    head_dense(net.W1, net.b1, net.in_dim, net.hidden_dim, relu, in, in_stride, tmp, tmp_stride, red);
    head_dense(net.W2, net.b2, net.hidden_dim, net.out_dim, relu && net.final_act, tmp, tmp_stride,
               out, out_stride, red);
}

// One block finishes kHeadStates states: chunk partial sums -> h_i -> head -> softmax.
__global__ void __launch_bounds__(kHeadThreads, 1)
pool_head_kernel(const PoolArgs a, int tmp_floats, int stage_floats) {
    extern __shared__ __align__(16) float smem[];
    const int d = a.d, F = a.F, B = a.B, m = a.m;
    const int E = 2 * d + F, Z = 5 * d + F;
    const int Zs = (Z + 3) & ~3;
    float *z = smem;                               // [states][Zs]
    float *sum = z + kHeadStates * Zs;             // [states][3 d]
    float *tmp = sum + kHeadStates * 3 * d;        // [states][tmp_floats]
    float *lg = tmp + kHeadStates * tmp_floats;    // [states][m]
    float *red = lg + ((kHeadStates * m + 3) & ~3);   // [blockDim.x * states] partial products
    const int b0 = blockIdx.x * kHeadStates;
    // The networks of this kernel: staged whole into shared memory with cp.async
    // when they fit (one round trip to L2 / DRAM instead of one per layer part),
    // otherwise read from global memory after an L2 prefetch.
    DevMlp net_h0 = a.h[0], net_h1 = a.h[1], net_h2 = a.h[2], net_head = a.head;
    if (stage_floats > 0) {
        float *w = red + (size_t)blockDim.x * kHeadStates;
        auto stage = [&](const float *&ptr, size_t count) {
            if (ptr == nullptr) return;
            if ((count & 3) == 0) {
                for (size_t i = (size_t)threadIdx.x * 4; i < count; i += (size_t)blockDim.x * 4)
                    __pipeline_memcpy_async(w + i, ptr + i, 16);
            } else {
                for (size_t i = threadIdx.x; i < count; i += blockDim.x)
                    __pipeline_memcpy_async(w + i, ptr + i, 4);
            }
            ptr = w;
            w += (count + 3) & ~size_t(3);
        };
        auto stage_net = [&](DevMlp &nt) {
            stage(nt.W1, (size_t)nt.in_dim * nt.hidden_dim);
            stage(nt.b1, nt.hidden_dim);
            if (nt.n_layers == 2) {
                stage(nt.W2, (size_t)nt.hidden_dim * nt.out_dim);
                stage(nt.b2, nt.out_dim);
            }
        };
        stage_net(net_h0);
        stage_net(net_h1);
        stage_net(net_h2);
        stage_net(net_head);
        __pipeline_commit();
    } else {
        prefetch_l2(a.head.W1, (size_t)a.head.in_dim * a.head.hidden_dim);
        if (a.head.n_layers == 2) prefetch_l2(a.head.W2, (size_t)a.head.hidden_dim * a.head.out_dim);
        for (int i = 0; i < 3; ++i) prefetch_l2(a.h[i].W1, (size_t)a.h[i].in_dim * a.h[i].hidden_dim);
    }
    dependency_wait();          // the partial sums come from a kernel that may still be running
    for (int i = threadIdx.x; i < kHeadStates * 3 * d; i += blockDim.x) {
        const int s = i / (3 * d), j = i - s * 3 * d;
        const int b = min(b0 + s, B - 1);          // rows past the batch repeat the last state
        // chunks are added in ascending order; four loads in flight at a time
        const float *src = a.partial + (size_t)b * 3 * d + j;
        const size_t step = (size_t)B * 3 * d;
        float acc = 0.f;
        int ch = 0;
        for (; ch + 4 <= a.chunks; ch += 4) {
            const float t0 = src[ch * step], t1 = src[(ch + 1) * step];
            const float t2 = src[(ch + 2) * step], t3 = src[(ch + 3) * step];
            acc = (((acc + t0) + t1) + t2) + t3;
        }
        for (; ch < a.chunks; ++ch) acc += src[ch * step];
        sum[i] = acc;
    }
    for (int i = threadIdx.x; i < kHeadStates * E; i += blockDim.x) {
        const int s = i / E, k = i - s * E;
        const int b = min(b0 + s, B - 1);
        const int c = a.cur[b];
        float v = 0.f;
        if (c >= 0 && c < a.n)
            v = k < d ? a.H[0][((size_t)c * B + b) * d + k]
              : k < 2 * d ? a.H[1][((size_t)c * B + b) * d + (k - d)]
                          : a.X[((size_t)c * B + b) * F + (k - 2 * d)];
        z[s * Zs + k] = v;
    }
    __pipeline_wait_prior(0);
    __syncthreads();
    if (net_h0.n_layers == 1 && net_h1.n_layers == 1 && net_h2.n_layers == 1) {
        // the three single-layer h_i in one pass: thread = (row, set, column)
        for (int i = threadIdx.x; i < kHeadStates * 3 * d; i += blockDim.x) {
            const int s = i / (3 * d), r = i - s * 3 * d;
            const int set = r / d, j = r - set * d;
            const DevMlp &nt = set == 0 ? net_h0 : (set == 1 ? net_h1 : net_h2);
            const float *v = sum + s * 3 * d + set * d;
            float a0 = nt.b1[j], a1 = 0.f;
            int k = 0;
            for (; k + 2 <= d; k += 2) {
                a0 = fmaf(v[k], nt.W1[(size_t)k * d + j], a0);
                a1 = fmaf(v[k + 1], nt.W1[(size_t)(k + 1) * d + j], a1);
            }
            if (k < d) a0 = fmaf(v[k], nt.W1[(size_t)k * d + j], a0);
            const float y = a0 + a1;
            z[s * Zs + E + r] = (nt.act == 0 && nt.final_act) ? fmaxf(y, 0.f) : y;
        }
        __syncthreads();
    } else {
        head_mlp(net_h0, sum, 3 * d, tmp, tmp_floats, z + E, Zs, red);
        head_mlp(net_h1, sum + d, 3 * d, tmp, tmp_floats, z + E + d, Zs, red);
        head_mlp(net_h2, sum + 2 * d, 3 * d, tmp, tmp_floats, z + E + 2 * d, Zs, red);
    }
    head_mlp(net_head, z, Zs, tmp, tmp_floats, lg, m, red);
    if (threadIdx.x < kHeadStates && b0 + threadIdx.x < B) {
        const int b = b0 + threadIdx.x;
        const float *l = lg + threadIdx.x * m;
        const int c = a.cur[b];
        // a current node out of range yields NaN (ReLU would swallow a NaN input)
        const bool valid = c >= 0 && c < a.n;
        float mx = l[0];
        for (int k = 1; k < m; ++k) mx = fmaxf(mx, l[k]);
        float tot = 0.f;
        for (int k = 0; k < m; ++k) tot += expf(l[k] - mx);
        for (int k = 0; k < m; ++k) {
            a.logits[(size_t)b * m + k] = valid ? l[k] : nanf("");
            if (a.probs) a.probs[(size_t)b * m + k] = valid ? expf(l[k] - mx) / tot : nanf("");
        }
    }
}

// The same finish for the common shapes (single-layer h_i of width d, two-layer
// head whose hidden width is a multiple of 4) with HS states per block, HS chosen
// so that the blocks cover the device: a small batch is spread over many SMs
// instead of eight states sharing one. Nothing is staged: weights are read once
// per block straight from L2 as 128-bit loads, a thread of the first head layer
// owns a (states x 4 columns) register tile and one part of the inner dimension,
// and activations sit transposed in shared memory ([k][state]) so that a tile's
// states come with one broadcast load. Parts are added in a fixed order.
constexpr int kFastThreads = 512;

template <int HS>
__global__ void __launch_bounds__(kFastThreads, 1)
pool_head_fast_kernel(const PoolArgs a) {
    constexpr int SR = HS < 4 ? HS : 4;     // states of a thread tile
    constexpr int SG = HS / SR;             // state groups
    extern __shared__ __align__(16) float smem[];
    const int d = a.d, F = a.F, B = a.B, m = a.m;
    const int E = 2 * d + F, Z = 5 * d + F, Hd = a.head.hidden_dim;
    float *zt = smem;                              // [Z][HS]: e_c, then the three h_i outputs
    float *sum = zt + Z * HS;                      // [HS][3 d]
    float *hid = sum + HS * 3 * d;                 // [Hd][HS]
    float *lg = hid + Hd * HS;                     // [HS][m]
    float *red = lg + ((HS * m + 3) & ~3);         // [parts][Hd][HS]
    const int b0 = blockIdx.x * HS;
    prefetch_l2(a.head.W1, (size_t)Z * Hd);
    prefetch_l2(a.head.W2, (size_t)Hd * m);
    for (int i = 0; i < 3; ++i) prefetch_l2(a.h[i].W1, (size_t)d * d);
    dependency_wait();          // the partial sums come from a kernel that may still be running
    for (int i = threadIdx.x; i < HS * 3 * d; i += blockDim.x) {
        const int s = i / (3 * d), j = i - s * 3 * d;
        const int b = min(b0 + s, B - 1);          // rows past the batch repeat the last state
        // chunks are added in ascending order; eight loads in flight at a time
        const float *src = a.partial + (size_t)b * 3 * d + j;
        const size_t step = (size_t)B * 3 * d;
        float acc = 0.f;
        for (int ch = 0; ch < a.chunks; ch += 8) {
            float t[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) t[q] = ch + q < a.chunks ? src[(ch + q) * step] : 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) acc += t[q];
        }
        sum[i] = acc;
    }
    for (int i = threadIdx.x; i < HS * E; i += blockDim.x) {
        const int s = i / E, k = i - s * E;
        const int b = min(b0 + s, B - 1);
        const int c = a.cur[b];
        float v = 0.f;
        if (c >= 0 && c < a.n)
            v = k < d ? a.H[0][((size_t)c * B + b) * d + k]
              : k < 2 * d ? a.H[1][((size_t)c * B + b) * d + (k - d)]
              : a.compact.state != nullptr ? compact_feature(a.compact, c, b, B, k - 2 * d)
                                           : a.X[((size_t)c * B + b) * F + (k - 2 * d)];
        zt[k * HS + s] = v;
    }
    __syncthreads();
    // the three h_i: thread = (state, set, four columns)
    const int dq = d >> 2;
    for (int i = threadIdx.x; i < HS * 3 * dq; i += blockDim.x) {
        const int s = i / (3 * dq), r = i - s * 3 * dq;
        const int set = r / dq, cq = r - set * dq;
        const DevMlp &nt = a.h[set];
        const float *__restrict__ W = nt.W1 + 4 * cq;
        const float *v = sum + s * 3 * d + set * d;
        float4 acc = *reinterpret_cast<const float4 *>(nt.b1 + 4 * cq);
        for (int kb = 0; kb < d; kb += 16) {   // sixteen weight rows in flight (d is a multiple of 4)
            float4 w[16];
#pragma unroll
            for (int t = 0; t < 16; ++t)
                w[t] = kb + t < d ? __ldg(reinterpret_cast<const float4 *>(W + (size_t)(kb + t) * d))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                const float x = kb + t < d ? v[kb + t] : 0.f;
                acc.x = fmaf(x, w[t].x, acc.x); acc.y = fmaf(x, w[t].y, acc.y);
                acc.z = fmaf(x, w[t].z, acc.z); acc.w = fmaf(x, w[t].w, acc.w);
            }
        }
        if (nt.act == 0 && nt.final_act) {
            acc.x = fmaxf(acc.x, 0.f); acc.y = fmaxf(acc.y, 0.f);
            acc.z = fmaxf(acc.z, 0.f); acc.w = fmaxf(acc.w, 0.f);
        }
        float *o = zt + (E + set * d + 4 * cq) * HS + s;
        o[0] = acc.x; o[HS] = acc.y; o[2 * HS] = acc.z; o[3 * HS] = acc.w;
    }
    __syncthreads();
    // head, first layer
    const int CG = Hd >> 2, tiles = SG * CG;
    const int parts = max(1, min((int)blockDim.x / tiles, Z));
    const int per = (Z + parts - 1) / parts;
    if ((int)threadIdx.x < tiles * parts) {
        const int part = threadIdx.x / tiles, r = threadIdx.x - part * tiles;
        const int sg = r / CG, cg = r - sg * CG;
        float acc[SR][4];
#pragma unroll
        for (int s = 0; s < SR; ++s)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[s][c] = 0.f;
        const int k0 = part * per, k1 = min(Z, k0 + per);
        const float *__restrict__ W = a.head.W1 + 4 * cg;
        const float *zrow = zt + sg * SR;
        for (int kb = k0; kb < k1; kb += 16) {   // sixteen weight rows in flight
            float4 w[16];
#pragma unroll
            for (int t = 0; t < 16; ++t)
                w[t] = kb + t < k1 ? __ldg(reinterpret_cast<const float4 *>(W + (size_t)(kb + t) * Hd))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                const bool live = kb + t < k1;
                const int k = live ? kb + t : k0;
                float zv[SR];
                if (SR == 4) {
                    const float4 u = *reinterpret_cast<const float4 *>(zrow + k * HS);
                    zv[0] = u.x; zv[1 % SR] = u.y; zv[2 % SR] = u.z; zv[3 % SR] = u.w;
                } else if (SR == 2) {
                    const float2 u = *reinterpret_cast<const float2 *>(zrow + k * HS);
                    zv[0] = u.x; zv[1 % SR] = u.y;
                } else {
                    zv[0] = zrow[k * HS];
                }
#pragma unroll
                for (int s = 0; s < SR; ++s) {
                    zv[s] = live ? zv[s] : 0.f;
                    acc[s][0] = fmaf(zv[s], w[t].x, acc[s][0]); acc[s][1] = fmaf(zv[s], w[t].y, acc[s][1]);
                    acc[s][2] = fmaf(zv[s], w[t].z, acc[s][2]); acc[s][3] = fmaf(zv[s], w[t].w, acc[s][3]);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int s = 0; s < SR; ++s)
                red[((size_t)part * Hd + 4 * cg + c) * HS + sg * SR + s] = acc[s][c];
    }
    __syncthreads();
    const bool relu = a.head.act == 0;
    for (int i = threadIdx.x; i < Hd * HS; i += blockDim.x) {
        float acc = a.head.b1[i / HS];
        for (int q = 0; q < parts; ++q) acc += red[(size_t)q * Hd * HS + i];
        hid[i] = relu ? fmaxf(acc, 0.f) : acc;
    }
    __syncthreads();
    // head, second layer: one warp per (state, device)
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
        for (int item = warp; item < HS * m; item += nw) {
            const int s = item / m, j = item - s * m;
            float acc = 0.f;
            for (int k = lane; k < Hd; k += 32) acc = fmaf(hid[k * HS + s], a.head.W2[(size_t)k * m + j], acc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            acc += a.head.b2[j];
            if (lane == 0) lg[s * m + j] = (relu && a.head.final_act) ? fmaxf(acc, 0.f) : acc;
        }
    }
    __syncthreads();
    if (threadIdx.x < HS && b0 + threadIdx.x < B) {
        const int b = b0 + threadIdx.x;
        const float *l = lg + threadIdx.x * m;
        const int c = a.cur[b];
        // a current node out of range yields NaN (ReLU would swallow a NaN input)
        const bool valid = c >= 0 && c < a.n;
        float mx = l[0];
        for (int k = 1; k < m; ++k) mx = fmaxf(mx, l[k]);
        float tot = 0.f;
        for (int k = 0; k < m; ++k) tot += expf(l[k] - mx);
        for (int k = 0; k < m; ++k) {
            a.logits[(size_t)b * m + k] = valid ? l[k] : nanf("");
            if (a.probs) a.probs[(size_t)b * m + k] = valid ? expf(l[k] - mx) / tot : nanf("");
        }
        if (a.step.enabled) {
            // The MDP transition of episode b (Sec. 2.1), fused here: greedy takes the largest
            // logit (lowest index among equals), sampling the first k with p_0 + .. + p_k > u for
            // p the FP32 softmax summed in index order (the last index if rounding leaves none).
            const EpisodeStep &st = a.step;
            int best = 0;
            float top = l[0];
            for (int k = 1; k < m; ++k)
                if (l[k] > top) { top = l[k]; best = k; }
            int action = best;
            if (st.uniforms != nullptr) {
                const float u = st.uniforms[(size_t)b * st.n + st.t];
                float cum = 0.f;
                action = m - 1;
                for (int k = 0; k < m; ++k) {
                    cum += expf(l[k] - mx) / tot;
                    if (cum > u) { action = k; break; }
                }
            }
            if (st.logp != nullptr) st.logp[(size_t)b * st.n + st.t] = (l[action] - mx) - logf(tot);
            if (st.actions != nullptr) st.actions[(size_t)b * st.n + st.t] = (uint8_t)action;
            const int v = st.order[st.t];
            if (v >= 0 && v < st.n) st.state[(size_t)v * B + b] = (uint8_t)(action | 0x80);   // placed, visited
            if (st.t + 1 < st.n) st.cur[b] = st.order[st.t + 1];
        }
    }
}

bool head_fast_applicable(const PoolArgs &a) {
    if ((a.d & 3) || a.head.n_layers != 2 || (a.head.hidden_dim & 3)) return false;
    if (a.head.hidden_dim / 4 * 2 > kFastThreads) return false;
    for (int i = 0; i < 3; ++i)
        if (a.h[i].n_layers != 1 || a.h[i].in_dim != a.d || a.h[i].out_dim != a.d) return false;
    return true;
}

template <int HS>
cudaError_t launch_head_fast(const PoolArgs &a, cudaStream_t stream) {
    const int Z = 5 * a.d + a.F, Hd = a.head.hidden_dim;
    constexpr int SR = HS < 4 ? HS : 4;
    const int tiles = (HS / SR) * (Hd / 4);
    const int parts = std::max(1, std::min(kFastThreads / tiles, Z));
    const size_t floats = (size_t)Z * HS + (size_t)HS * 3 * a.d + (size_t)Hd * HS + ((HS * a.m + 3) & ~3) +
                          (size_t)parts * Hd * HS;
    const size_t bytes = floats * sizeof(float);
    if (bytes > 200 * 1024) return cudaErrorNotSupported;
    cudaError_t err = cudaFuncSetAttribute(pool_head_fast_kernel<HS>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (err != cudaSuccess) return err;
    // always preceded by one of this library's pooling kernels on the same stream
    err = launch_overlapped(true, pool_head_fast_kernel<HS>, dim3((a.B + HS - 1) / HS), dim3(kFastThreads),
                            bytes, stream, a);
    count_launch();
    return err;
}

}  // namespace

bool pool_head_takes_compact(const PoolArgs &a) { return head_fast_applicable(a); }

int pool_chunks(int n, int B, const DeviceInfo &di) {
    // enough (chunk, state-group) blocks to fill the device a few times over
    const int state_blocks = (B + kPoolWarps - 1) / kPoolWarps;
    int chunks = (4 * di.sm_count + state_blocks - 1) / state_blocks;
    chunks = std::max(1, std::min(chunks, (n + 7) / 8));
    return chunks;
}

cudaError_t launch_policy_generic(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream) {
    PoolPlan p;
    const int E = 2 * a.d + a.F;
    int max_hidden = 0;
    size_t wfloats = 0;
    for (int i = 0; i < 3; ++i) {
        const DevMlp &m = a.l[i];
        if (m.n_layers == 2) max_hidden = std::max(max_hidden, m.hidden_dim);
        wfloats += (((size_t)m.in_dim * m.hidden_dim + 3) & ~size_t(3)) + ((m.hidden_dim + 3) & ~3);
        if (m.n_layers == 2)
            wfloats += (((size_t)m.hidden_dim * m.out_dim + 3) & ~size_t(3)) + ((m.out_dim + 3) & ~3);
    }
    p.e_stride = ((E + 3) & ~3) + ((max_hidden + 3) & ~3);
    const size_t rows_bytes = (size_t)kPoolWarps * p.e_stride * sizeof(float);
    const size_t budget = (size_t)std::min(di.max_smem_optin, 200 * 1024);
    p.weights_in_smem = (wfloats * sizeof(float) + rows_bytes <= budget) ? 1 : 0;
    p.smem_bytes = rows_bytes + (p.weights_in_smem ? wfloats * sizeof(float) : 0);
    p.states_per_block = kPoolWarps;
    cudaError_t err = cudaFuncSetAttribute(pool_partial_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    dim3 grid(a.chunks, (a.B + p.states_per_block - 1) / p.states_per_block);
    pool_partial_kernel<<<grid, kPoolThreads, p.smem_bytes, stream>>>(a, p);
    count_launch();
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    return launch_pool_head(a, di, stream);
}

cudaError_t launch_pool_head(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream) {
    if (head_fast_applicable(a)) {
        // fewest states per block that keeps the grid within two blocks per SM
        const int limit = 2 * std::max(1, di.sm_count);
        cudaError_t e = (a.B + 1) / 2 <= limit   ? launch_head_fast<2>(a, stream)
                        : (a.B + 3) / 4 <= limit ? launch_head_fast<4>(a, stream)
                                                 : launch_head_fast<8>(a, stream);
        if (e != cudaErrorNotSupported) return e;
    }
    const int Z = 5 * a.d + a.F;
    int tmp_floats = a.head.n_layers == 2 ? a.head.hidden_dim : 0;
    for (int i = 0; i < 3; ++i)
        if (a.h[i].n_layers == 2) tmp_floats = std::max(tmp_floats, a.h[i].hidden_dim);
    tmp_floats = (tmp_floats + 3) & ~3;
    size_t head_smem =
        ((size_t)kHeadStates * (((Z + 3) & ~3) + 3 * a.d + tmp_floats + a.m) + 4 +
         (size_t)kHeadThreads * kHeadStates) * sizeof(float);
    // floats of all networks, each array padded to a multiple of 4
    size_t stage_floats = 0;
    for (const DevMlp *nt : {&a.h[0], &a.h[1], &a.h[2], &a.head}) {
        stage_floats += (((size_t)nt->in_dim * nt->hidden_dim + 3) & ~size_t(3)) + ((nt->hidden_dim + 3) & ~3);
        if (nt->n_layers == 2)
            stage_floats += (((size_t)nt->hidden_dim * nt->out_dim + 3) & ~size_t(3)) + ((nt->out_dim + 3) & ~3);
    }
    if (head_smem + stage_floats * sizeof(float) <= 200 * 1024) head_smem += stage_floats * sizeof(float);
    else stage_floats = 0;
    cudaError_t err = cudaFuncSetAttribute(pool_head_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)head_smem);
    if (err != cudaSuccess) return err;
    const int blocks = (a.B + kHeadStates - 1) / kHeadStates;
    // always preceded by one of this library's pooling kernels on the same stream
    err = launch_overlapped(true, pool_head_kernel, dim3(blocks), dim3(kHeadThreads), head_smem, stream, a,
                            tmp_floats, (int)stage_floats);
    count_launch();
    return err;
}

}  // namespace placeto
