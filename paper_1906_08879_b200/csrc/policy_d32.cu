// Step 3 of the policy (Sec. 2.2 step 3 of the Placeto paper) specialised for
// d = 32 with single-layer ReLU l_i: the per-set sums
//   sum_{u in S_i(c)} l_i(e_u),   e_u = [h_down_u || h_up_u || x_u],
// for a chunk of nodes and a tile of 16 states per block, written as partial
// sums that the head kernel adds up in chunk order.
//
// A block first copies its whole tile (chunk x 16 states of H_down, H_up, X) and
// the three weight matrices into shared memory with bulk asynchronous copies
// (one per matrix, three per node, counted on an mbarrier). Warp w owns state
// w of the tile. For each set i in turn it loads column `lane` of W_i into
// registers, scans the relation row of its state's current node over the chunk
// (ballot), and pushes the rows of set i through the 32 x (64 + F) product two at
// a time, reading the inputs as broadcast 128-bit shared loads; the sums stay in
// registers. Summation order is ascending node id: deterministic.
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 32;
constexpr int kWarps = 16;             // = states per block
constexpr int kThreads = kWarps * 32;

struct Pool32Plan {
    int chunk_nodes, chunks;
    size_t smem_bytes;
};

typedef unsigned long long pair_t;   // two FP32 values in one 64-bit register pair

__device__ __forceinline__ pair_t pack2(float lo, float hi) {
    pair_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ float sum2(pair_t v) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}
// two independent FP32 FMAs in one instruction (sm_100 packed arithmetic)
__device__ __forceinline__ pair_t fma2(pair_t a, pair_t b, pair_t c) {
    pair_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// acc[r] += in[r][0..K) . w for R rows; w holds the column as pairs (w[2i], w[2i+1]),
// every 128-bit shared load feeds two packed FMAs.
template <int R, int K>
__device__ __forceinline__ void fma_rows(const pair_t *w, const float *const (&in)[R],
                                         pair_t (&acc)[R][2]) {
#pragma unroll
    for (int k = 0; k < K; k += 4) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const ulonglong2 u = *reinterpret_cast<const ulonglong2 *>(in[r] + k);
            acc[r][0] = fma2(u.x, w[k / 2], acc[r][0]);
            acc[r][1] = fma2(u.y, w[k / 2 + 1], acc[r][1]);
        }
    }
}

template <int F4, bool kCompact>     // kCompact: the raw features come from compact states, not from X
__global__ void __launch_bounds__(kThreads, 1)
pool_d32_kernel(const PoolArgs a, const Pool32Plan p) {
    constexpr int FP = 4 * F4;             // padded feature width
    constexpr int E = 2 * kD + FP;
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = a.n, B = a.B, F = a.F;
    const int chunk = blockIdx.x;
    const int u0 = chunk * p.chunk_nodes, nu = min(n, u0 + p.chunk_nodes) - u0;
    const int b0 = blockIdx.y * kWarps, nb = min(kWarps, B - b0);

    float *Ws = smem;                                   // [3][E][32], rows past 64 + F are zero
    float *bs = Ws + 3 * E * kD;                        // [3][32]
    float *hd = bs + 3 * kD;                            // [chunk][16][32]
    float *hu = hd + (size_t)p.chunk_nodes * kWarps * kD;
    float *xs = hu + (size_t)p.chunk_nodes * kWarps * kD;   // [chunk][16][FP]

    // ---- stage weights and the tile: one bulk copy per matrix and three per node
    // (16 states x 32 floats of H_down and H_up, 16 states x F of X are contiguous
    // both in global and in shared memory), all reporting to one mbarrier
    __shared__ __align__(8) unsigned long long bar;
    const unsigned w_bytes = (unsigned)(E * kD * sizeof(float));      // F == FP here: no padding rows
    const unsigned h_bytes = (unsigned)(nb * kD * sizeof(float)), x_bytes = (unsigned)(nb * F * sizeof(float));
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_expect(&bar, 3 * w_bytes + (unsigned)nu * (2 * h_bytes + (kCompact ? 0u : x_bytes)));
    }
    if (threadIdx.x < 3 * kD) bs[threadIdx.x] = a.l[threadIdx.x / kD].b1[threadIdx.x % kD];
    __syncthreads();
    if (threadIdx.x == 0)
        for (int i = 0; i < 3; ++i) bulk_load(Ws + i * E * kD, a.l[i].W1, w_bytes, &bar);
    dependency_wait();          // the embeddings may come from a kernel that is still running
    for (int t = threadIdx.x; t < 3 * nu; t += kThreads) {
        const int q = t / 3, which = t - 3 * q;
        const size_t row = (size_t)(u0 + q) * B + b0;
        if (which == 0) bulk_load(hd + (size_t)q * kWarps * kD, a.H[0] + row * kD, h_bytes, &bar);
        else if (which == 1) bulk_load(hu + (size_t)q * kWarps * kD, a.H[1] + row * kD, h_bytes, &bar);
        else if (!kCompact) bulk_load(xs + (size_t)q * kWarps * FP, a.X + row * F, x_bytes, &bar);
    }
    if (kCompact) {
        // no X tensor: the tile's features from one byte per (node, state)
        for (int i = threadIdx.x; i < nu * nb; i += kThreads) {     // one (node, state) pair per thread
            const int q = i / nb, st = i - q * nb;
            compact_features(a.compact, u0 + q, b0 + st, B, xs + (size_t)q * kWarps * FP + st * FP);
        }
        __syncthreads();
    }
    const bool landed = mbar_wait(&bar, 0);
    if (!landed && threadIdx.x == 0) report_status(a.status, PLACETO_ERR_TIMEOUT);

    if (warp >= nb) return;
    const int b = b0 + warp;
    const int c = a.cur[b];
    const bool valid = c >= 0 && c < n;
    PLACETO_DEBUG_CHECK(a.status, valid);
    const uint8_t *rel = a.relation + (size_t)(valid ? c : 0) * n + u0;
    float *out = a.partial + ((size_t)chunk * B + b) * 3 * kD;
    for (int i = 0; i < 3; ++i) {
        pair_t w[E / 2];
#pragma unroll
        for (int k = 0; k < E; k += 2)
            w[k / 2] = pack2(Ws[(i * E + k) * kD + lane], Ws[(i * E + k + 1) * kD + lane]);
        const float bias = bs[i * kD + lane];
        float total = 0.f;
        for (int base = 0; base < nu && valid; base += 32) {
            const int q = base + lane;
            unsigned mask = __ballot_sync(0xffffffffu, q < nu && rel[q] == i);
            while (mask) {
                const int qa = base + __ffs(mask) - 1;
                mask &= mask - 1;
                if (mask) {
                    const int qb = base + __ffs(mask) - 1;
                    mask &= mask - 1;
                    pair_t acc[2][2] = {{pack2(bias, 0.f), 0ull}, {pack2(bias, 0.f), 0ull}};
                    const size_t ra = (size_t)qa * kWarps + warp, rb = (size_t)qb * kWarps + warp;
                    const float *const pd[2] = {hd + ra * kD, hd + rb * kD};
                    const float *const pu[2] = {hu + ra * kD, hu + rb * kD};
                    const float *const px[2] = {xs + ra * FP, xs + rb * FP};
                    fma_rows<2, kD>(w, pd, acc);
                    fma_rows<2, kD>(w + kD / 2, pu, acc);
                    fma_rows<2, FP>(w + kD, px, acc);
                    total += fmaxf(sum2(acc[0][0]) + sum2(acc[0][1]), 0.f);
                    total += fmaxf(sum2(acc[1][0]) + sum2(acc[1][1]), 0.f);
                } else {
                    pair_t acc[1][2] = {{pack2(bias, 0.f), 0ull}};
                    const size_t ra = (size_t)qa * kWarps + warp;
                    const float *const pd[1] = {hd + ra * kD};
                    const float *const pu[1] = {hu + ra * kD};
                    const float *const px[1] = {xs + ra * FP};
                    fma_rows<1, kD>(w, pd, acc);
                    fma_rows<1, kD>(w + kD / 2, pu, acc);
                    fma_rows<1, FP>(w + kD, px, acc);
                    total += fmaxf(sum2(acc[0][0]) + sum2(acc[0][1]), 0.f);
                }
            }
        }
        out[i * kD + lane] = landed ? total : nanf("");   // a copy that never landed shows as NaN logits
    }
}

bool relu1(const DevMlp &m, int in) {
    return m.n_layers == 1 && m.in_dim == in && m.out_dim == kD && m.act == 0 && m.final_act == 1;
}

}  // namespace

bool pool_d32_applicable(const PoolArgs &a) {
    if (a.d != kD || a.F < 4 || a.F > 16 || (a.F & 3)) return false;
    for (int i = 0; i < 3; ++i)
        if (!relu1(a.l[i], 2 * kD + a.F)) return false;
    return true;
}

// Nodes per chunk and number of chunks for a batch of B states.
void pool_d32_chunks(int n, int B, int F, const DeviceInfo &di, int *chunk_nodes, int *chunks) {
    const int E = 2 * kD + F;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    const size_t fixed = (size_t)(3 * E * kD + 3 * kD) * sizeof(float);
    const size_t per_node = (size_t)kWarps * E * sizeof(float);
    const int cap = std::max(1, (int)((budget - fixed) / per_node));
    const int tiles = (B + kWarps - 1) / kWarps;
    int c = (n + cap - 1) / cap;
    // a single wave: give every SM a block if the chunks can be made smaller
    if (c * tiles < di.sm_count) c = std::max(c, std::min(di.sm_count / tiles, (n + 7) / 8));
    c = std::max(1, c);
    *chunk_nodes = (n + c - 1) / c;
    *chunks = (n + *chunk_nodes - 1) / *chunk_nodes;
}

bool pool_d32_fits(const PoolArgs &a, const DeviceInfo &di) {
    const int E = 2 * kD + a.F;
    const size_t bytes = ((size_t)(3 * E * kD + 3 * kD) + (size_t)a.chunk_nodes * kWarps * E) * sizeof(float);
    return pool_d32_applicable(a) && a.chunk_nodes > 0 && bytes <= (size_t)di.max_smem_optin;
}

cudaError_t launch_pool_d32(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream,
                            bool overlap) {
    Pool32Plan p;
    p.chunk_nodes = a.chunk_nodes;
    p.chunks = a.chunks;
    const int E = 2 * kD + a.F;
    p.smem_bytes = ((size_t)(3 * E * kD + 3 * kD) + (size_t)p.chunk_nodes * kWarps * E) * sizeof(float);
    if (p.smem_bytes > (size_t)di.max_smem_optin) return cudaErrorNotSupported;
    void (*kern)(const PoolArgs, const Pool32Plan) = nullptr;
    switch (a.F / 4) {
        case 1: kern = a.compact.state ? pool_d32_kernel<1, true> : pool_d32_kernel<1, false>; break;
        case 2: kern = a.compact.state ? pool_d32_kernel<2, true> : pool_d32_kernel<2, false>; break;
        case 3: kern = a.compact.state ? pool_d32_kernel<3, true> : pool_d32_kernel<3, false>; break;
        case 4: kern = a.compact.state ? pool_d32_kernel<4, true> : pool_d32_kernel<4, false>; break;
        default: return cudaErrorNotSupported;
    }
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    dim3 grid(p.chunks, (a.B + kWarps - 1) / kWarps);
    err = launch_overlapped(overlap, kern, grid, dim3(kThreads), p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace placeto
