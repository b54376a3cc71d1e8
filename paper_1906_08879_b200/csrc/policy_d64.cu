// Step 3 of the policy (Sec. 2.2 step 3 of the Placeto paper) specialised for
// d = 64 with single-layer ReLU l_i: partial sums over a chunk of nodes of
//   l_i(e_u),   e_u = [h_down_u || h_up_u || x_u],   i = set of u relative to cur[b],
// for a tile of states per block, in the layout the head kernel adds up.
//
// The block works one set at a time: lane (quarter, pair) keeps two adjacent
// columns of W_i for one quarter of the inner dimension (2 x 36 registers), four
// warps cover the 64 columns, and the two groups of four warps take alternate
// states of the tile. A warp reads its quarter of a row from shared memory (one
// address per quarter-warp, the cheapest pattern of a 128-bit load, feeding 8
// FMAs per lane), combines the quarters with two shuffles per column and adds
// relu(.) to the sum of the (state, set) list it is walking. A row is read by
// four warps instead of the eight that one column per lane needs. The rows of
// each (state, set) are compacted into index lists while the tile is staged
// (bulk asynchronous copies), so the main loop runs list by list, two rows in
// flight, without branching on the set. Warps never synchronise after staging.
// Summation order is ascending node id per (chunk, state, set): deterministic.
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 64;
constexpr int kWarps = kD / 8;
constexpr int kThreads = kWarps * 32;
constexpr int kTileStates = 8;

struct Pool64Plan {
    int chunk_nodes, chunks;
    size_t smem_bytes;
};

constexpr int kCols = 4;      // adjacent output columns per lane

// Sum over one set's rows (node indices in `list`) of relu(bias + row . w) for this
// lane's columns; two rows in flight, two accumulators per row and column.
template <int KQ, int RS>
__device__ __forceinline__ void set_sum(const float (&w)[kCols][KQ], const float (&bias)[kCols],
                                        const uint8_t *list, int count, const float *rows_s,
                                        float (&total)[kCols]) {
#pragma unroll
    for (int c = 0; c < kCols; ++c) total[c] = 0.f;
    for (int i = 0; i < count; i += 2) {
        const bool two = i + 1 < count;
        const float *in0 = rows_s + (size_t)list[i] * (kTileStates * RS);
        const float *in1 = rows_s + (size_t)list[two ? i + 1 : i] * (kTileStates * RS);
        float a[2][kCols][2];
#pragma unroll
        for (int r = 0; r < 2; ++r)
#pragma unroll
            for (int c = 0; c < kCols; ++c) a[r][c][0] = a[r][c][1] = 0.f;
#pragma unroll
        for (int k = 0; k < KQ; k += 4) {
            const float4 u = *reinterpret_cast<const float4 *>(in0 + k);
            const float4 v = *reinterpret_cast<const float4 *>(in1 + k);
#pragma unroll
            for (int c = 0; c < kCols; ++c) {
                a[0][c][0] = fmaf(u.x, w[c][k], a[0][c][0]);     a[1][c][0] = fmaf(v.x, w[c][k], a[1][c][0]);
                a[0][c][1] = fmaf(u.y, w[c][k + 1], a[0][c][1]); a[1][c][1] = fmaf(v.y, w[c][k + 1], a[1][c][1]);
                a[0][c][0] = fmaf(u.z, w[c][k + 2], a[0][c][0]); a[1][c][0] = fmaf(v.z, w[c][k + 2], a[1][c][0]);
                a[0][c][1] = fmaf(u.w, w[c][k + 3], a[0][c][1]); a[1][c][1] = fmaf(v.w, w[c][k + 3], a[1][c][1]);
            }
        }
#pragma unroll
        for (int c = 0; c < kCols; ++c) {
            float t0 = a[0][c][0] + a[0][c][1], t1 = a[1][c][0] + a[1][c][1];
            t0 += __shfl_xor_sync(0xffffffffu, t0, 8);         // the four quarters of the inner dimension
            t1 += __shfl_xor_sync(0xffffffffu, t1, 8);
            t0 += __shfl_xor_sync(0xffffffffu, t0, 16);
            t1 += __shfl_xor_sync(0xffffffffu, t1, 16);
            total[c] += fmaxf(t0 + bias[c], 0.f);
            if (two) total[c] += fmaxf(t1 + bias[c], 0.f);
        }
    }
}

template <int F4>
__global__ void __launch_bounds__(kThreads, 1)
pool_d64_kernel(const PoolArgs a, const Pool64Plan p) {
    constexpr int E = 2 * kD + 4 * F4;              // embedding row (features padded to 4 F4)
    constexpr int KQ = ((E + 3) / 4 + 3) & ~3;      // inner width per lane quarter
    constexpr int RS = 4 * KQ;                      // shared row stride (>= E, zero padded)
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    dependency_wait();          // the embeddings may come from a kernel that is still running
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // four groups of two warps each cover all 64 columns (32 per warp, four per lane) and share
    // the tile's states between them; a lane keeps a quarter of the inner dimension
    constexpr int kGroups = kWarps / 2;
    const int quarter = lane >> 3, col = (warp & 1) * 32 + kCols * (lane & 7), group = warp >> 1;
    const int n = a.n, B = a.B, F = a.F;
    const int chunk = blockIdx.x;
    const int u0 = chunk * p.chunk_nodes, nu = min(n, u0 + p.chunk_nodes) - u0;
    const int b0 = blockIdx.y * kTileStates, nb = min(kTileStates, B - b0);

    float *rows = smem;                                                    // [chunk][states][RS]
    // per state and set: the chunk's node indices of that set, ascending  [states][3][chunk]
    uint8_t *lists = reinterpret_cast<uint8_t *>(rows + (size_t)p.chunk_nodes * kTileStates * RS);
    __shared__ int counts[kTileStates][3];
    // ---- stage the tile: every row as one contiguous [h_down | h_up | x | 0] vector,
    // three bulk copies per (node, state) row reporting to one mbarrier
    __shared__ __align__(8) unsigned long long bar;
    {
        const unsigned x_bytes = (unsigned)(F * sizeof(float)), h_bytes = (unsigned)(kD * sizeof(float));
        if (threadIdx.x == 0) {
            mbar_init(&bar, 1);
            mbar_expect(&bar, (unsigned)(nu * nb) * (2 * h_bytes + x_bytes));
        }
        __syncthreads();
        for (int t = threadIdx.x; t < nu * nb * 3; t += kThreads) {
            const int r = t / 3, which = t - 3 * r;
            const int q = r / nb, s = r - q * nb;
            const size_t src = (size_t)(u0 + q) * B + b0 + s;
            float *dst = rows + ((size_t)q * kTileStates + s) * RS;
            if (which == 0) bulk_load(dst, a.H[0] + src * kD, h_bytes, &bar);
            else if (which == 1) bulk_load(dst + kD, a.H[1] + src * kD, h_bytes, &bar);
            else bulk_load(dst + 2 * kD, a.X + src * F, x_bytes, &bar);
        }
        const int pad = RS - (2 * kD + F);
        for (int t = threadIdx.x; t < nu * nb * pad; t += kThreads) {
            const int r = t / pad, k = t - r * pad;
            const int q = r / nb, s = r - q * nb;
            rows[((size_t)q * kTileStates + s) * RS + 2 * kD + F + k] = 0.f;
        }
    }
    if (warp < nb) {       // warp s compacts the relation row of its state into three lists
        const int c = a.cur[b0 + warp];
        const bool valid = c >= 0 && c < n;
    PLACETO_DEBUG_CHECK(a.status, valid);
        const uint8_t *rel = a.relation + (size_t)(valid ? c : 0) * n + u0;
        int cnt[3] = {0, 0, 0};
        for (int base = 0; base < nu; base += 32) {
            const int q = base + lane;
            const int set = (valid && q < nu) ? rel[q] : 3;
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const unsigned mask = __ballot_sync(0xffffffffu, set == i);
                if (set == i)
                    lists[(warp * 3 + i) * p.chunk_nodes + cnt[i] + __popc(mask & ((1u << lane) - 1))] =
                        (uint8_t)q;
                cnt[i] += __popc(mask);
            }
        }
        if (lane < 3) counts[warp][lane] = lane == 0 ? cnt[0] : (lane == 1 ? cnt[1] : cnt[2]);
    }
    // ---- one set at a time: this lane's four columns of W_i, its quarter of the inner dimension
    float w[kCols][KQ];
    auto load_set = [&](int i) {
#pragma unroll
        for (int k = 0; k < KQ; ++k) {
            const int kk = quarter * KQ + k;
            const float4 v = kk < 2 * kD + F ? *reinterpret_cast<const float4 *>(a.l[i].W1 + kk * kD + col)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
            w[0][k] = v.x; w[1][k] = v.y; w[2][k] = v.z; w[3][k] = v.w;
        }
    };
    load_set(0);
    const bool landed = mbar_wait(&bar, 0);
    if (!landed && threadIdx.x == 0) report_status(a.status, PLACETO_ERR_TIMEOUT);
    __syncthreads();            // lists, counts and the zero padding written by other threads

    for (int i = 0; i < 3; ++i) {
        const float4 b4 = *reinterpret_cast<const float4 *>(a.l[i].b1 + col);
        const float bias[kCols] = {b4.x, b4.y, b4.z, b4.w};
        for (int s = group; s < nb; s += kGroups) {
            const float *rows_s = rows + (size_t)s * RS + quarter * KQ;
            const uint8_t *ls = lists + ((size_t)s * 3 + i) * p.chunk_nodes;
            float acc[kCols];
            set_sum<KQ, RS>(w, bias, ls, counts[s][i], rows_s, acc);
            if (quarter == 0) {
                // a copy that never landed shows as NaN logits
                float *out = a.partial + ((size_t)chunk * B + b0 + s) * 3 * kD + i * kD + col;
                const float bad = nanf("");
                *reinterpret_cast<float4 *>(out) = landed ? make_float4(acc[0], acc[1], acc[2], acc[3])
                                                          : make_float4(bad, bad, bad, bad);
            }
        }
        if (i < 2) load_set(i + 1);
    }
}

bool relu1x64(const DevMlp &m, int in) {
    return m.n_layers == 1 && m.in_dim == in && m.out_dim == kD && m.act == 0 && m.final_act == 1;
}

size_t tile_bytes(int chunk_nodes, int F) {
    const int E = 2 * kD + F;
    const int KQ = ((E + 3) / 4 + 3) & ~3;
    return (size_t)chunk_nodes * kTileStates * 4 * KQ * sizeof(float) +
           (((size_t)chunk_nodes * kTileStates * 3 + 15) & ~size_t(15));
}

}  // namespace

bool pool_d64_applicable(const PoolArgs &a) {
    if (a.d != kD || a.F < 4 || a.F > 16 || (a.F & 3)) return false;
    for (int i = 0; i < 3; ++i)
        if (!relu1x64(a.l[i], 2 * kD + a.F)) return false;
    return true;
}

void pool_d64_chunks(int n, int B, int F, const DeviceInfo &di, int *chunk_nodes, int *chunks) {
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    int cap = 1;
    while (cap < 255 && tile_bytes(cap + 1, F) <= budget) ++cap;
    const int tiles = (B + kTileStates - 1) / kTileStates;
    int c = (n + cap - 1) / cap;
    if (c * tiles < di.sm_count) c = std::max(c, std::min(di.sm_count / tiles, (n + 7) / 8));
    c = std::max(1, c);
    *chunk_nodes = (n + c - 1) / c;
    *chunks = (n + *chunk_nodes - 1) / *chunk_nodes;
}

cudaError_t launch_pool_d64(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream,
                            bool overlap) {
    Pool64Plan p;
    p.chunk_nodes = a.chunk_nodes;
    p.chunks = a.chunks;
    p.smem_bytes = tile_bytes(p.chunk_nodes, a.F);
    // node indices inside a chunk are stored as bytes
    if (p.smem_bytes > (size_t)di.max_smem_optin || p.chunk_nodes > 255) return cudaErrorNotSupported;
    void (*kern)(const PoolArgs, const Pool64Plan) = nullptr;
    switch (a.F / 4) {
        case 1: kern = pool_d64_kernel<1>; break;
        case 2: kern = pool_d64_kernel<2>; break;
        case 3: kern = pool_d64_kernel<3>; break;
        case 4: kern = pool_d64_kernel<4>; break;
        default: return cudaErrorNotSupported;
    }
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    dim3 grid(p.chunks, (a.B + kTileStates - 1) / kTileStates);
    err = launch_overlapped(overlap, kern, grid, dim3(kThreads), p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace placeto
