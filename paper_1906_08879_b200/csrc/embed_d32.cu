// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper) specialised for
// embedding width d = 32 with two-layer ReLU networks of hidden width 32:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]).
//
// Design (one block = one direction x one slice of the state batch, walking all
// levels with __syncthreads() between levels; states never interact):
//   - Lane j of every warp keeps column j of all four weight matrices of the
//     direction in registers (32 + 32 + (32 + F) + 32 values), so a warp carries
//     a row (node, state) through gather -> g1 -> g2 -> f1 -> f2 on its own.
//     Between layers the 32 outputs are exchanged through a per-warp shared
//     buffer and read back as broadcast 128-bit loads: 4 FMAs per shared load,
//     issued as two packed fma.rn.f32x2 against weights kept in register pairs.
//   - Two states of a node are in flight per warp (one on narrow levels), with
//     four dependent accumulator chains per row.
//   - Messages never leave the SM: m_u lives in a shared-memory slot from the
//     level of u until its last consumer's level (slots assigned on the host).
//     Global traffic is the compulsory part only: read x, write h.
//   - The level schedule (order, CSR, slots) is staged in shared memory, and the
//     raw features of the next level are copied asynchronously (cp.async) into a
//     double-buffered staging area while the current level computes, so no DRAM
//     latency sits on the level-to-level critical path.
#include <cuda_pipeline.h>

#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 32;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

struct D32Plan {
    int S;          // states per slice
    int n_slices;
    int x_floats;   // floats of one feature staging buffer (widest level x S x F, padded)
    size_t smem_bytes;
};

typedef unsigned long long pair_t;   // two FP32 values in one 64-bit register pair

__device__ __forceinline__ pair_t pack2(float lo, float hi) {
    pair_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2(pair_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// Two independent FP32 FMAs in one instruction (sm_100 packed arithmetic): half
// the FMA issue slots, the same rounding as two fmaf.
__device__ __forceinline__ pair_t fma2(pair_t a, pair_t b, pair_t c) {
    pair_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// out[r] = bias + in[r] . w for R rows whose K inputs are read as broadcast
// 128-bit loads from shared memory. The weights are kept as pairs (w[2i],
// w[2i + 1]) so that every load feeds two packed FMAs; two pair accumulators per
// row, i.e. four dependent chains of K / 4 FMAs.
template <int R, int K>
__device__ __forceinline__ void matvec(const pair_t (&w)[K / 2], float bias, const float *in,
                                       int row_stride, float (&out)[R]) {
    pair_t acc[R][2];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        acc[r][0] = pack2(bias, 0.f);
        acc[r][1] = 0ull;
    }
#pragma unroll
    for (int k = 0; k < K; k += 4) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const ulonglong2 u = *reinterpret_cast<const ulonglong2 *>(in + r * row_stride + k);
            acc[r][0] = fma2(u.x, w[k / 2], acc[r][0]);
            acc[r][1] = fma2(u.y, w[k / 2 + 1], acc[r][1]);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float a, b, c, d;
        unpack2(acc[r][0], a, b);
        unpack2(acc[r][1], c, d);
        out[r] = (a + b) + (c + d);
    }
}

struct Weights32 {
    pair_t g1[kD / 2], g2[kD / 2], f2[kD / 2];   // column `lane`, rows in pairs
    float bg1, bg2, bf1, bf2;
};

// Carries R states (s0 .. s0 + R - 1 of the slice; the last may be missing and
// then repeats s0) of the node at position `pos` through
// gather -> g -> store h -> f -> store m. The R rows share the node, so the
// schedule lookups are done once. A, Bf: the warp's exchange buffers, R rows of
// KF floats each. All shared-memory offsets are 32-bit.
template <int R, int KF>
__device__ __forceinline__ void run_node(const Weights32 &w, const pair_t (&wf1)[KF / 2], int pos,
                                         int q, int s0, bool last_live, int nb, int S, int F,
                                         int lane, const int4 *meta, const int *nbr_slot,
                                         float *msg, const float *xs, float *__restrict__ H,
                                         size_t B, int b_first, float *A, float *Bf) {
    int st[R];
    float x[R], acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        st[r] = (r == 0 || last_live) ? s0 + r : s0;
        x[r] = lane < F ? xs[(q * nb + st[r]) * F + lane] : 0.f;
        acc[r] = 0.f;
    }
    const int4 m = meta[pos];       // {first neighbour entry, end, own | first neighbour slot, node}
    const int e1 = m.y, v = m.w;
    const int slot = (m.z & 0xffff) == 0xffff ? -1 : (m.z & 0xffff);
    int e = m.x;
    if (e1 - e == 1) {
        // One neighbour (most nodes of chain-like graphs): its message row is the
        // input of g as it stands, so the first layer reads the slot directly and
        // the gather, the store and the warp barrier are skipped.
        const float *row = msg + ((int)((unsigned)m.z >> 16) * S + st[0]) * kD;
        matvec<R, kD>(w.g1, w.bg1, row, (R > 1 && last_live) ? kD : 0, acc);
        __syncwarp();               // the previous node's last reads of Bf are done
        goto after_g1;
    }
    for (; e + 4 <= e1; e += 4) {   // four neighbours at a time: the loads overlap
        int base[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) base[k] = nbr_slot[e + k] * S;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float t[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) t[k] = msg[(base[k] + st[r]) * kD + lane];
            acc[r] += (t[0] + t[1]) + (t[2] + t[3]);
        }
    }
    for (; e < e1; ++e) {
        const int base = nbr_slot[e] * S;
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] += msg[(base + st[r]) * kD + lane];
    }
#pragma unroll
    for (int r = 0; r < R; ++r) A[r * KF + lane] = acc[r];
    __syncwarp();
    matvec<R, kD>(w.g1, w.bg1, A, KF, acc);
after_g1:
#pragma unroll
    for (int r = 0; r < R; ++r) Bf[r * KF + lane] = fmaxf(acc[r], 0.f);
    __syncwarp();
    matvec<R, kD>(w.g2, w.bg2, Bf, KF, acc);
    float *hrow = H + ((size_t)v * B + b_first + s0) * kD + lane;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        acc[r] = fmaxf(acc[r], 0.f);
        if (r == 0 || last_live) hrow[r * kD] = acc[r];
    }
    if (slot < 0) return;                   // nobody consumes this node's message
#pragma unroll
    for (int r = 0; r < R; ++r) {
        A[r * KF + lane] = acc[r];
        if (lane < KF - kD) A[r * KF + kD + lane] = x[r];
    }
    __syncwarp();
    matvec<R, KF>(wf1, w.bf1, A, KF, acc);
#pragma unroll
    for (int r = 0; r < R; ++r) Bf[r * KF + lane] = fmaxf(acc[r], 0.f);
    __syncwarp();
    matvec<R, kD>(w.f2, w.bf2, Bf, KF, acc);
#pragma unroll
    for (int r = 0; r < R; ++r)
        if (r == 0 || last_live) msg[((slot * S) + st[r]) * kD + lane] = fmaxf(acc[r], 0.f);
}

template <int F4, bool kCompact>   // feature width padded to 4 * F4; features built from compact states
__global__ void __launch_bounds__(kThreads, 1)
embed_d32_kernel(const EmbedArgs a, const D32Plan p) {
    constexpr int KF = kD + 4 * F4;      // padded input width of f's first layer
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    const int dir = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F;
    const int b_first = blockIdx.x * p.S;
    const int nb = min(p.S, B - b_first);

    // ---- shared memory: [schedule ints][message slots][feature staging x2][exchange buffers]
    // one packed record per position: {first neighbour entry, end,
    // own slot (low 16 bits, 0xffff = none) | slot of the first neighbour (high 16 bits), node id}
    int4 *meta_w = reinterpret_cast<int4 *>(smem);
    for (int i = threadIdx.x; i < a.n; i += kThreads) {
        const int e0 = lv.nbr_ptr[i], e1 = lv.nbr_ptr[i + 1];
        const int first = e1 > e0 ? lv.nbr_slot[e0] : 0;
        meta_w[i] = make_int4(e0, e1, (lv.own_slot[i] & 0xffff) | (first << 16), lv.order[i]);
        PLACETO_DEBUG_CHECK(a.status, e0 >= 0 && e0 <= e1 && e1 <= lv.n_nbr && lv.own_slot[i] >= -1 &&
                                          lv.own_slot[i] < lv.n_slots && lv.order[i] >= 0 && lv.order[i] < a.n);
    }
    for (int e = threadIdx.x; e < lv.n_nbr; e += kThreads)
        PLACETO_DEBUG_CHECK(a.status, lv.nbr_slot[e] >= 0 && lv.nbr_slot[e] < lv.n_slots);
    PLACETO_DEBUG_CHECK(a.status, nb >= 1 && b_first + nb <= B);
    const int4 *meta = meta_w;
    int *ism = reinterpret_cast<int *>(smem) + 4 * a.n;
    auto stage = [&](const int *src, int count) {
        int *dst = ism;
        for (int i = threadIdx.x; i < count; i += kThreads) dst[i] = src[i];
        ism += (count + 3) & ~3;
        return (const int *)dst;
    };
    const int *level_ptr = stage(lv.level_ptr, lv.n_levels + 1);
    const int *nbr_slot = stage(lv.nbr_slot, lv.n_nbr);
    float *fsm = reinterpret_cast<float *>(ism);
    float *msg = fsm;                                       // [n_slots][S][32]
    float *xstage = msg + (size_t)lv.n_slots * p.S * kD;    // [2][x_floats]
    float *xbuf = xstage + 2 * (size_t)p.x_floats + (size_t)warp * 4 * KF;
    float *A = xbuf, *Bf = xbuf + 2 * KF;

    // ---- this lane's weight columns
    const DevMlp f = a.f[dir], g = a.g[dir];
    Weights32 w;
    pair_t wf1[KF / 2];
#pragma unroll
    for (int k = 0; k < kD; k += 2) {
        w.g1[k / 2] = pack2(g.W1[k * kD + lane], g.W1[(k + 1) * kD + lane]);
        w.g2[k / 2] = pack2(g.W2[k * kD + lane], g.W2[(k + 1) * kD + lane]);
        w.f2[k / 2] = pack2(f.W2[k * kD + lane], f.W2[(k + 1) * kD + lane]);
    }
#pragma unroll
    for (int k = 0; k < KF; k += 2)
        wf1[k / 2] = pack2(k < kD + F ? f.W1[k * kD + lane] : 0.f,
                           k + 1 < kD + F ? f.W1[(k + 1) * kD + lane] : 0.f);
    w.bg1 = g.b1[lane]; w.bg2 = g.b2[lane]; w.bf1 = f.b1[lane]; w.bf2 = f.b2[lane];
    const float *__restrict__ X = a.X;
    float *__restrict__ H = a.H[dir];
    __syncthreads();

    // Asynchronous copy of one level's raw features (rows of the slice) into a
    // staging buffer, so that the next level's x is on chip when it is needed.
    // exact division of small non-negative numbers by a per-block constant
    auto magic_of = [](int d) { return (unsigned)((0x100000000ull + d - 1) / d); };
    const unsigned magic_nb = magic_of(nb), magic_ppn = magic_of((nb + 1) >> 1);
    const int per_node = nb * F;             // floats per node, contiguous in X
    const bool vec = (F & 3) == 0;
    const int per = vec ? per_node >> 2 : per_node;     // copy pieces per node
    const unsigned magic_per = magic_of(per);
    // The last warp (the one least often needed for rows) issues all copies, so
    // the other warps go straight to their rows.
    auto prefetch = [&](int level) {
        if (warp != kWarps - 1) return;
        const int q0 = level_ptr[level], width = level_ptr[level + 1] - q0;
        float *dst = xstage + (size_t)(level & 1) * p.x_floats;
        if (kCompact) {
            // no X tensor: the level's features from one byte per (node, state)
            for (int i = lane; i < width * nb; i += 32) {       // one (node, state) pair per lane
                const int q = nb == 1 ? i : (int)__umulhi((unsigned)i, magic_nb), s = i - q * nb;
                compact_features(a.compact, meta[q0 + q].w, b_first + s, (int)B, dst + (size_t)i * F);
            }
            return;
        }
        for (int i = lane; i < width * per; i += 32) {
            const int q = per == 1 ? i : (int)__umulhi((unsigned)i, magic_per);
            const int piece = i - q * per;
            const float *src = X + ((size_t)meta[q0 + q].w * B + b_first) * F;
            if (vec) __pipeline_memcpy_async(dst + q * per_node + 4 * piece, src + 4 * piece, 16);
            else __pipeline_memcpy_async(dst + q * per_node + piece, src + piece, 4);
        }
        __pipeline_commit();
    };
    dependency_wait();          // the raw features may come from a kernel that is still running
    prefetch(0);
    __pipeline_wait_prior(0);
    __syncthreads();

    for (int level = 0; level < lv.n_levels; ++level) {
        if (level + 1 < lv.n_levels) prefetch(level + 1);
        const int p0 = level_ptr[level];
        const int rows = (level_ptr[level + 1] - p0) * nb;
        const float *xs = xstage + (size_t)(level & 1) * p.x_floats;
        const int width = level_ptr[level + 1] - p0;
        if (rows <= kWarps) {
            // narrow level: one row per warp, shortest dependent chains
            if (warp < rows) {
                const int q = nb == 1 ? warp : (int)__umulhi((unsigned)warp, magic_nb);
                const int s0 = warp - q * nb;
                run_node<1, KF>(w, wf1, p0 + q, q, s0, true, nb, p.S, F, lane, meta, nbr_slot, msg,
                                xs, H, B, b_first, A, Bf);
            }
        } else {
            // two states of one node per warp pass
            const int ppn = (nb + 1) >> 1;
            for (int item = warp; item < width * ppn; item += kWarps) {
                const int q = ppn == 1 ? item : (int)__umulhi((unsigned)item, magic_ppn);
                const int s0 = (item - q * ppn) * 2;
                run_node<2, KF>(w, wf1, p0 + q, q, s0, s0 + 1 < nb, nb, p.S, F, lane, meta, nbr_slot,
                                msg, xs, H, B, b_first, A, Bf);
            }
        }
        __pipeline_wait_prior(0);
        __syncthreads();
    }
}

bool relu2x32(const DevMlp &m, int in) {
    return m.n_layers == 2 && m.in_dim == in && m.hidden_dim == kD && m.out_dim == kD &&
           m.act == 0 && m.final_act == 1;
}

}  // namespace

bool embed_d32_applicable(const EmbedArgs &a) {
    if (a.d != kD || a.F < 1 || a.F > 16) return false;
    for (int dir = 0; dir < 2; ++dir)
        if (!relu2x32(a.f[dir], kD + a.F) || !relu2x32(a.g[dir], kD)) return false;
    return true;
}

namespace {
// slice size and shared-memory layout; false when not even one state per block fits
bool plan_d32(const EmbedArgs &a, const DeviceInfo &di, D32Plan *out) {
    D32Plan p;
    const int target = std::max(1, di.sm_count / 2);            // blocks per direction
    const int want = std::max(1, std::min(a.B, target));
    p.S = (a.B + want - 1) / want;
    const int F4 = (a.F + 3) / 4;
    const int KF = kD + 4 * F4;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    const int max_slots = std::max(a.lv[0].n_slots, a.lv[1].n_slots);
    if (max_slots >= 0xffff) return false;   // slot ids are packed into 16 bits
    size_t ints = 0;
    for (int dir = 0; dir < 2; ++dir) {
        const DevLevels &lv = a.lv[dir];
        ints = std::max(ints, (size_t)4 * a.n + ((lv.n_levels + 1 + 3) & ~3) + ((lv.n_nbr + 3) & ~3));
    }
    const size_t xbuf = (size_t)kWarps * 4 * KF * sizeof(float);
    auto x_floats = [&](int S) { return (a.max_level_width * S * a.F + 3) & ~3; };
    auto need = [&](int S) {
        return (size_t)max_slots * S * kD * sizeof(float) + 2 * (size_t)x_floats(S) * sizeof(float) +
               xbuf + ints * sizeof(int);
    };
    // narrower slices when the shared memory does not fit (more blocks: they queue up)
    while (p.S > 1 && need(p.S) > budget) --p.S;
    if (need(p.S) > budget) return false;
    // more slices than one wave of blocks: spread the batch evenly over the waves it takes
    {
        const int waves = ((a.B + p.S - 1) / p.S + want - 1) / want;
        p.S = std::min(p.S, (a.B + want * waves - 1) / (want * waves));
    }
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.x_floats = x_floats(p.S);
    p.smem_bytes = need(p.S);
    *out = p;
    return true;
}
}  // namespace

bool embed_d32_fits(const EmbedArgs &a, const DeviceInfo &di) {
    D32Plan p;
    return embed_d32_applicable(a) && plan_d32(a, di, &p);
}

cudaError_t launch_embed_d32(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream,
                             bool overlap) {
    D32Plan p;
    if (!plan_d32(a, di, &p)) return cudaErrorNotSupported;
    const int F4 = (a.F + 3) / 4;
    void (*kern)(const EmbedArgs, const D32Plan) = nullptr;
    const bool compact = a.compact.state != nullptr;
    switch (F4) {
        case 1: kern = compact ? embed_d32_kernel<1, true> : embed_d32_kernel<1, false>; break;
        case 2: kern = compact ? embed_d32_kernel<2, true> : embed_d32_kernel<2, false>; break;
        case 3: kern = compact ? embed_d32_kernel<3, true> : embed_d32_kernel<3, false>; break;
        case 4: kern = compact ? embed_d32_kernel<4, true> : embed_d32_kernel<4, false>; break;
        default: return cudaErrorNotSupported;
    }
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    err = launch_overlapped(overlap, kern, dim3(p.n_slices, 2), dim3(kThreads), p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace placeto
