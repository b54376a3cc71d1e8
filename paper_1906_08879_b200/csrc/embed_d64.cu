// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper) specialised for
// embedding width d = 64 with two-layer ReLU networks of hidden width 64:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]).
//
// At d = 64 one direction's weights (17 K floats) do not fit in one warp's
// registers, so four warps form a group that owns a direction: warp c of the
// group keeps output columns [16c, 16c + 16) of all four matrices, lane
// (half, col) holding one half of the inner dimension of its column (about 136
// registers). A layer is: every lane reads its half of the input rows from the
// group's shared exchange buffer (broadcast 128-bit loads), multiplies, the two
// halves are combined with one shuffle, and the 64 outputs are exchanged through
// shared memory with a 128-thread named barrier. Four states of a node are in
// flight per group. A block runs both directions (two groups) for one slice of
// the state batch and walks all levels without any grid-wide sync; the groups
// never wait for each other.
//
// As in the d = 32 kernel, messages stay in shared-memory slots assigned on the
// host, the level schedule is staged in shared memory and the next level's raw
// features are fetched with cp.async while the current level computes.
#include <cuda_pipeline.h>

#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 64;
constexpr int kGroupWarps = 4;
constexpr int kGroupThreads = kGroupWarps * 32;
constexpr int kThreads = 2 * kGroupThreads;
constexpr int kR = 4;                 // states of one node in flight per group

struct D64Plan {
    int S, n_slices;
    int x_floats;                     // floats of one feature staging buffer
    int int_floats[2];                // shared-memory floats taken by each direction's schedule
    size_t smem_bytes;
};

__device__ __forceinline__ void group_sync(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "n"(kGroupThreads) : "memory");
}

// part[r] = sum over this lane's half of the inner dimension, for kR rows.
template <int KH>
__device__ __forceinline__ void half_dot(const float (&w)[KH], const float *in, int row_stride,
                                         float (&out)[kR]) {
    float acc[kR][2];
#pragma unroll
    for (int r = 0; r < kR; ++r) acc[r][0] = acc[r][1] = 0.f;
#pragma unroll
    for (int k = 0; k < KH; k += 4) {
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            const float4 u = *reinterpret_cast<const float4 *>(in + r * row_stride + k);
            acc[r][0] = fmaf(u.x, w[k], acc[r][0]);
            acc[r][1] = fmaf(u.y, w[k + 1], acc[r][1]);
            acc[r][0] = fmaf(u.z, w[k + 2], acc[r][0]);
            acc[r][1] = fmaf(u.w, w[k + 3], acc[r][1]);
        }
    }
#pragma unroll
    for (int r = 0; r < kR; ++r) {
        const float s = acc[r][0] + acc[r][1];
        out[r] = s + __shfl_xor_sync(0xffffffffu, s, 16);      // add the other half
    }
}

template <int F4>
__global__ void __launch_bounds__(kThreads, 1)
embed_d64_kernel(const EmbedArgs a, const D64Plan p) {
    constexpr int KF = kD + 4 * F4;                 // input width of f's first layer (padded)
    constexpr int KH = ((KF + 1) / 2 + 3) & ~3;     // per-half inner width of that layer
    constexpr int KP = 2 * KH;                      // exchange row stride
    extern __shared__ __align__(16) float smem[];
    const int group = threadIdx.x / kGroupThreads;  // 0 top-down, 1 bottom-up
    const int gt = threadIdx.x - group * kGroupThreads;
    const int warp = gt >> 5, lane = gt & 31;
    const int half = lane >> 4, col = warp * 16 + (lane & 15);
    const DevLevels lv = a.lv[group];
    const int B = a.B, F = a.F, S = p.S;
    const int b_first = blockIdx.x * S;
    const int nb = min(S, B - b_first);

    // ---- shared memory, per group: [schedule ints][message slots][x staging x2][exchange A, B]
    float *base = smem;
    if (group == 1)
        base += p.int_floats[0] + (size_t)a.lv[0].n_slots * S * kD + 2 * (size_t)p.x_floats + 2 * kR * KP;
    int *ism = reinterpret_cast<int *>(base);
    auto stage = [&](const int *src, int count) {
        int *dst = ism;
        for (int i = gt; i < count; i += kGroupThreads) dst[i] = src[i];
        ism += (count + 3) & ~3;
        return (const int *)dst;
    };
    const int *level_ptr = stage(lv.level_ptr, lv.n_levels + 1);
    const int *order = stage(lv.order, a.n);
    const int *nbr_ptr = stage(lv.nbr_ptr, a.n + 1);
    const int *own_slot = stage(lv.own_slot, a.n);
    const int *nbr_slot = stage(lv.nbr_slot, lv.n_nbr);
    float *msg = base + p.int_floats[group];                    // [n_slots][S][64]
    float *xstage = msg + (size_t)lv.n_slots * S * kD;          // [2][x_floats]
    float *A = xstage + 2 * (size_t)p.x_floats;                 // [kR][KP]
    float *Bf = A + kR * KP;                                    // [kR][KP]

    // ---- this lane's weights: column `col`, inner indices of its half
    const DevMlp f = a.f[group], g = a.g[group];
    float wg1[kD / 2], wg2[kD / 2], wf2[kD / 2], wf1[KH];
#pragma unroll
    for (int k = 0; k < kD / 2; ++k) {
        const int kk = half * (kD / 2) + k;
        wg1[k] = g.W1[kk * kD + col];
        wg2[k] = g.W2[kk * kD + col];
        wf2[k] = f.W2[kk * kD + col];
    }
#pragma unroll
    for (int k = 0; k < KH; ++k) {
        const int kk = half * KH + k;
        wf1[k] = kk < kD + F ? f.W1[kk * kD + col] : 0.f;
    }
    const float bg1 = g.b1[col], bg2 = g.b2[col], bf1 = f.b1[col], bf2 = f.b2[col];
    const float *__restrict__ X = a.X;
    float *__restrict__ H = a.H[group];

    const int per_node = nb * F;
    auto prefetch = [&](int level) {
        const int q0 = level_ptr[level], width = level_ptr[level + 1] - q0;
        float *dst = xstage + (size_t)(level & 1) * p.x_floats;
        if ((F & 3) == 0) {
            const int per = per_node >> 2;
            for (int i = gt; i < width * per; i += kGroupThreads) {
                const int q = i / per, off = (i - q * per) * 4;
                __pipeline_memcpy_async(dst + q * per_node + off,
                                        X + ((size_t)order[q0 + q] * B + b_first) * F + off, 16);
            }
        } else {
            for (int i = gt; i < width * per_node; i += kGroupThreads) {
                const int q = i / per_node, off = i - q * per_node;
                __pipeline_memcpy_async(dst + i, X + ((size_t)order[q0 + q] * B + b_first) * F + off, 4);
            }
        }
        __pipeline_commit();
    };
    group_sync(group);            // schedule staged
    prefetch(0);
    __pipeline_wait_prior(0);
    group_sync(group);

    const int batches = (nb + kR - 1) / kR;      // state batches per node
    for (int level = 0; level < lv.n_levels; ++level) {
        if (level + 1 < lv.n_levels) prefetch(level + 1);
        const int p0 = level_ptr[level], width = level_ptr[level + 1] - p0;
        const float *xs = xstage + (size_t)(level & 1) * p.x_floats;
        for (int item = 0; item < width * batches; ++item) {
            const int q = item / batches, s0 = (item - q * batches) * kR;
            const int pos = p0 + q;
            const int live = min(kR, nb - s0);              // states of this batch that exist
            const int e0 = nbr_ptr[pos], e1 = nbr_ptr[pos + 1];
            const int slot = own_slot[pos];
            const int v = order[pos];
            // rows this lane finishes (bias, activation, stores): r = half and half + 2
            int st[2];
#pragma unroll
            for (int t = 0; t < 2; ++t) st[t] = s0 + min(half + 2 * t, live - 1);
            // gather: sum of the neighbours' messages, this lane's column, its two rows
            float s[2] = {0.f, 0.f};
            for (int e = e0; e < e1; ++e) {
                const int mb = nbr_slot[e] * S;
#pragma unroll
                for (int t = 0; t < 2; ++t) s[t] += msg[(mb + st[t]) * kD + col];
            }
#pragma unroll
            for (int t = 0; t < 2; ++t) A[(half + 2 * t) * KP + col] = s[t];
            group_sync(group);
            float acc[kR];
            half_dot<kD / 2>(wg1, A + half * (kD / 2), KP, acc);
#pragma unroll
            for (int t = 0; t < 2; ++t) Bf[(half + 2 * t) * KP + col] = fmaxf((half ? acc[2 * t + 1] : acc[2 * t]) + bg1, 0.f);
            group_sync(group);
            half_dot<kD / 2>(wg2, Bf + half * (kD / 2), KP, acc);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int r = half + 2 * t;
                const float h = fmaxf((half ? acc[2 * t + 1] : acc[2 * t]) + bg2, 0.f);
                if (r < live) H[((size_t)v * B + b_first + s0 + r) * kD + col] = h;
                A[r * KP + col] = h;
            }
            if (slot >= 0) {                                 // group-uniform: somebody reads the message
                // raw features and zero padding behind the 64 embedding columns
                for (int i = gt; i < kR * (KP - kD); i += kGroupThreads) {
                    const int r = i / (KP - kD), k = i - r * (KP - kD);
                    const int sr = s0 + min(r, live - 1);
                    A[r * KP + kD + k] = k < F ? xs[(q * nb + sr) * F + k] : 0.f;
                }
                group_sync(group);
                half_dot<KH>(wf1, A + half * KH, KP, acc);
#pragma unroll
                for (int t = 0; t < 2; ++t) Bf[(half + 2 * t) * KP + col] = fmaxf((half ? acc[2 * t + 1] : acc[2 * t]) + bf1, 0.f);
                group_sync(group);
                half_dot<kD / 2>(wf2, Bf + half * (kD / 2), KP, acc);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int r = half + 2 * t;
                    if (r < live)
                        msg[(slot * S + s0 + r) * kD + col] =
                            fmaxf((half ? acc[2 * t + 1] : acc[2 * t]) + bf2, 0.f);
                }
            }
            // the next item writes A again: everyone must be done reading it
            group_sync(group);
        }
        __pipeline_wait_prior(0);
        group_sync(group);
    }
}

bool relu2x64(const DevMlp &m, int in) {
    return m.n_layers == 2 && m.in_dim == in && m.hidden_dim == kD && m.out_dim == kD &&
           m.act == 0 && m.final_act == 1;
}

}  // namespace

bool embed_d64_applicable(const EmbedArgs &a) {
    if (a.d != kD || a.F < 1 || a.F > 16) return false;
    for (int dir = 0; dir < 2; ++dir)
        if (!relu2x64(a.f[dir], kD + a.F) || !relu2x64(a.g[dir], kD)) return false;
    return true;
}

cudaError_t launch_embed_d64(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream) {
    D64Plan p;
    const int want = std::max(1, std::min(a.B, di.sm_count));
    p.S = (a.B + want - 1) / want;
    const int F4 = (a.F + 3) / 4;
    const int KF = kD + 4 * F4;
    const int KH = ((KF + 1) / 2 + 3) & ~3;
    const int KP = 2 * KH;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    for (int dir = 0; dir < 2; ++dir) {
        const DevLevels &lv = a.lv[dir];
        p.int_floats[dir] = ((lv.n_levels + 1 + 3) & ~3) + 2 * ((a.n + 3) & ~3) + ((a.n + 1 + 3) & ~3) +
                            ((lv.n_nbr + 3) & ~3);
    }
    auto x_floats = [&](int S) { return (a.max_level_width * S * a.F + 3) & ~3; };
    auto need = [&](int S) {
        size_t floats = 0;
        for (int dir = 0; dir < 2; ++dir)
            floats += (size_t)p.int_floats[dir] + (size_t)a.lv[dir].n_slots * S * kD +
                      2 * (size_t)x_floats(S) + 2 * (size_t)kR * KP;
        return floats * sizeof(float);
    };
    while (p.S > 1 && need(p.S) > budget) --p.S;
    if (need(p.S) > budget) return cudaErrorNotSupported;
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.x_floats = x_floats(p.S);
    p.smem_bytes = need(p.S);
    void (*kern)(const EmbedArgs, const D64Plan) = nullptr;
    switch (F4) {
        case 1: kern = embed_d64_kernel<1>; break;
        case 2: kern = embed_d64_kernel<2>; break;
        case 3: kern = embed_d64_kernel<3>; break;
        case 4: kern = embed_d64_kernel<4>; break;
        default: return cudaErrorNotSupported;
    }
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    kern<<<p.n_slices, kThreads, p.smem_bytes, stream>>>(a, p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace placeto
