// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper) on the tensor
// cores, for d = 32 and d = 64 with two-layer ReLU networks of hidden width d:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]).
//
// The kernels that keep weights in registers and broadcast activations from
// shared memory deliver two operands per lane per shared-memory wavefront and
// are therefore capped at half the FP32 FMA rate. Here a level's rows (node,
// state) of one block are packed into 16-row tiles and every layer is a
// 16 x K x d product on mma.sync.m16n8k8 (TF32 inputs, FP32 accumulate). To keep
// FP32 accuracy each operand is split into a TF32 head and a TF32 tail and three
// products are accumulated (head*head + head*tail + tail*head); the dropped
// tail*tail term is below 2^-22 relative.
//
// Work split: a group of d/8 warps owns one direction; warp w of the group owns
// output columns [8w, 8w + 8) of all four matrices and keeps them, split into
// head and tail, as B fragments in registers. The 16 x K activation tile travels
// between layers through a padded row-major shared buffer (conflict-free
// fragment loads) with a named barrier per layer. As in the other kernels,
// messages live in shared-memory slots assigned on the host, the level schedule
// is staged in shared memory, and the next level's raw features arrive by
// cp.async while the current level computes. A block owns a slice of the state
// batch and walks all levels without grid-wide synchronisation; at d = 32 it runs
// both directions (two groups), at d = 64 one direction (blockIdx.y).
#include <cuda_pipeline.h>

#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kTile = 16;

struct MmaPlan {
    int S, n_slices;
    int x_floats;          // floats of one feature staging buffer
    int int_floats[2];     // shared-memory floats taken by each direction's schedule
    size_t smem_bytes;
};

__device__ __forceinline__ unsigned tf32_of(float x) {
    unsigned r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

// Round-to-nearest (ties away from zero) to TF32 with two integer operations:
// the conversion instruction runs at a fraction of the ALU rate and, issued
// eight times per k-step, was the bottleneck of the layer loop.
__device__ __forceinline__ unsigned tf32_round(float x) {
    return (__float_as_uint(x) + 0x1000u) & 0xffffe000u;
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], const unsigned (&a)[4], unsigned b0,
                                         unsigned b1) {
    asm(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// One warp's B fragments (head and tail) of a K x 8 column block: for k-step ks,
// b0 = W[8 ks + t][n0 + g], b1 = W[8 ks + t + 4][n0 + g] with g = lane / 4, t = lane % 4.
template <int NKS>
struct BFrag {
    unsigned h0[NKS], h1[NKS], l0[NKS], l1[NKS];
    __device__ __forceinline__ void load(const float *W, int ld, int n_rows, int n0, int lane) {
        const int g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int ks = 0; ks < NKS; ++ks) {
            const int k0 = 8 * ks + t, k1 = k0 + 4;
            const float w0 = k0 < n_rows ? W[(size_t)k0 * ld + n0 + g] : 0.f;
            const float w1 = k1 < n_rows ? W[(size_t)k1 * ld + n0 + g] : 0.f;
            h0[ks] = tf32_of(w0);
            h1[ks] = tf32_of(w1);
            l0[ks] = tf32_of(w0 - __uint_as_float(h0[ks]));
            l1[ks] = tf32_of(w1 - __uint_as_float(h1[ks]));
        }
    }
};

// Splits two adjacent activations into TF32 head and tail and stores both (the
// producer of a value splits it once; every consuming warp loads the halves).
__device__ __forceinline__ void store_split(float *head, int tail_offset, float x, float y) {
    const unsigned hx = tf32_round(x), hy = tf32_round(y);
    *reinterpret_cast<float2 *>(head) = make_float2(__uint_as_float(hx), __uint_as_float(hy));
    *reinterpret_cast<float2 *>(head + tail_offset) =
        make_float2(__uint_as_float(tf32_round(x - __uint_as_float(hx))),
                    __uint_as_float(tf32_round(y - __uint_as_float(hy))));
}

// c = tile (16 x 8 NKS: TF32 heads row-major in shared memory with row stride P,
// the tails in a second array of the same shape right behind) times this warp's
// column block, in the C-fragment layout:
//   c[0], c[1] = (row g,     cols 2t, 2t + 1);  c[2], c[3] = (row g + 8, same cols).
template <int NKS>
__device__ __forceinline__ void tile_product(const BFrag<NKS> &b, const float *buf, int P, int lane,
                                             float (&c)[4]) {
    // The legacy MMA path has a long dependent-issue latency (about 110 cycles
    // measured), so the k-steps accumulate into independent chains: one chain
    // per k-step up to four, two k-steps per chain beyond.
    constexpr int NCH = NKS <= 4 ? NKS : (NKS + 1) / 2;
    const int g = lane >> 2, t = lane & 3;
    float hh[NCH][4], hl[NCH][4], lh[NCH][4];
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
        for (int i = 0; i < 4; ++i) hh[ch][i] = hl[ch][i] = lh[ch][i] = 0.f;
    const float *h0 = buf + g * P + t, *h1 = buf + (g + 8) * P + t;
    const float *l0 = h0 + kTile * P, *l1 = h1 + kTile * P;      // tails follow the heads
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
        const unsigned ah[4] = {__float_as_uint(h0[8 * ks]), __float_as_uint(h1[8 * ks]),
                                __float_as_uint(h0[8 * ks + 4]), __float_as_uint(h1[8 * ks + 4])};
        const unsigned al[4] = {__float_as_uint(l0[8 * ks]), __float_as_uint(l1[8 * ks]),
                                __float_as_uint(l0[8 * ks + 4]), __float_as_uint(l1[8 * ks + 4])};
        mma_tf32(lh[ks % NCH], al, b.h0[ks], b.h1[ks]);
        mma_tf32(hl[ks % NCH], ah, b.l0[ks], b.l1[ks]);
        mma_tf32(hh[ks % NCH], ah, b.h0[ks], b.h1[ks]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float small = 0.f, big = 0.f;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            small += hl[ch][i] + lh[ch][i];
            big += hh[ch][i];
        }
        c[i] = big + small;
    }
}

template <int D, int NKF>   // NKF: k-steps of f's first layer, 8 NKF >= D + F
__global__ void __launch_bounds__(256, 1)
embed_mma_kernel(const EmbedArgs a, const MmaPlan p) {
    constexpr int GW = D / 8;                       // warps per group
    constexpr int GT = GW * 32;                     // threads per group
    constexpr int KF = 8 * NKF;                     // padded input width of f's first layer
    constexpr int P = KF + 4;                       // exchange row stride (P mod 8 == 4)
    constexpr int NKD = D / 8;
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    const int group = threadIdx.x / GT;             // d = 32: 0 top-down, 1 bottom-up
    const int dir = D == 32 ? group : (int)blockIdx.y;
    const int gt = threadIdx.x - group * GT;
    const int warp = gt >> 5, lane = gt & 31;
    const int g = lane >> 2, t = lane & 3;
    const int c0 = 8 * warp + 2 * t;                // this lane's two output columns
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F, S = p.S;
    const int b_first = blockIdx.x * S;
    const int nb = min(S, B - b_first);
    const int bar_id = group + 1;
    auto group_sync = [&]() {
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(GT) : "memory");
    };

    // ---- shared memory per group: [schedule][message slots][x staging x2][tile A, tile B: head+tail]
    float *base = smem;
    if (D == 32 && group == 1)
        base += p.int_floats[0] + (size_t)a.lv[0].n_slots * S * D + 2 * (size_t)p.x_floats + 4 * kTile * P;
    // level_ptr, nbr_slot and one packed record per position:
    //   meta[p] = {first neighbour entry, end of neighbour entries, own slot, node id}
    int *ism = reinterpret_cast<int *>(base);
    int4 *meta_w = reinterpret_cast<int4 *>(ism);
    for (int i = gt; i < a.n; i += GT)
    {
        meta_w[i] = make_int4(lv.nbr_ptr[i], lv.nbr_ptr[i + 1], lv.own_slot[i], lv.order[i]);
        PLACETO_DEBUG_CHECK(a.status, lv.nbr_ptr[i] >= 0 && lv.nbr_ptr[i] <= lv.nbr_ptr[i + 1] &&
                                          lv.nbr_ptr[i + 1] <= lv.n_nbr && lv.own_slot[i] >= -1 &&
                                          lv.own_slot[i] < lv.n_slots && lv.order[i] >= 0 && lv.order[i] < a.n);
    }
    for (int e = gt; e < lv.n_nbr; e += GT)
        PLACETO_DEBUG_CHECK(a.status, lv.nbr_slot[e] >= 0 && lv.nbr_slot[e] < lv.n_slots);
    PLACETO_DEBUG_CHECK(a.status, nb >= 1 && b_first + nb <= B);
    ism += 4 * a.n;
    auto stage = [&](const int *src, int count) {
        int *dst = ism;
        for (int i = gt; i < count; i += GT) dst[i] = src[i];
        ism += (count + 3) & ~3;
        return (const int *)dst;
    };
    const int4 *meta = meta_w;
    const int *level_ptr = stage(lv.level_ptr, lv.n_levels + 1);
    const int *nbr_slot = stage(lv.nbr_slot, lv.n_nbr);
    float *msg = base + p.int_floats[dir];                      // [n_slots][S][D]
    float *xstage = msg + (size_t)lv.n_slots * S * D;           // [2][x_floats]
    float *bufA = xstage + 2 * (size_t)p.x_floats;              // heads [16][P], tails [16][P]
    float *bufB = bufA + 2 * kTile * P;                         // the same for the other parity
    constexpr int TAIL = kTile * P;

    // ---- this warp's weights as B fragments, biases for its two columns
    const DevMlp f = a.f[dir], gm = a.g[dir];
    BFrag<NKD> wg1, wg2, wf2;
    BFrag<NKF> wf1;
    wg1.load(gm.W1, D, D, 8 * warp, lane);
    wg2.load(gm.W2, D, D, 8 * warp, lane);
    wf1.load(f.W1, D, D + F, 8 * warp, lane);
    wf2.load(f.W2, D, D, 8 * warp, lane);
    const float2 bg1 = make_float2(gm.b1[c0], gm.b1[c0 + 1]), bg2 = make_float2(gm.b2[c0], gm.b2[c0 + 1]);
    const float2 bf1 = make_float2(f.b1[c0], f.b1[c0 + 1]), bf2 = make_float2(f.b2[c0], f.b2[c0 + 1]);
    const float *__restrict__ X = a.X;
    float *__restrict__ H = a.H[dir];

    // exact division of small non-negative numbers by a per-block constant
    auto magic_of = [](int d) { return (unsigned)((0x100000000ull + d - 1) / d); };
    const unsigned magic_nb = magic_of(nb);
    const int per_node = nb * F;
    const bool vec = (F & 3) == 0;
    const int per = vec ? per_node >> 2 : per_node;     // copy pieces per node
    const unsigned magic_per = magic_of(per);
    auto prefetch = [&](int level) {
        const int q0 = level_ptr[level], width = level_ptr[level + 1] - q0;
        float *dst = xstage + (size_t)(level & 1) * p.x_floats;
        for (int i = gt; i < width * per; i += GT) {
            const int q = per == 1 ? i : (int)__umulhi((unsigned)i, magic_per);
            const int piece = i - q * per;
            const float *src = X + ((size_t)meta[q0 + q].w * B + b_first) * F;
            if (vec) __pipeline_memcpy_async(dst + q * per_node + 4 * piece, src + 4 * piece, 16);
            else __pipeline_memcpy_async(dst + q * per_node + piece, src + piece, 4);
        }
        __pipeline_commit();
    };
    group_sync();                 // schedule staged
    dependency_wait();            // the raw features may come from a kernel that is still running
    prefetch(0);
    __pipeline_wait_prior(0);
    group_sync();

    for (int level = 0; level < lv.n_levels; ++level) {
        if (level + 1 < lv.n_levels) prefetch(level + 1);
        const int p0 = level_ptr[level];
        const int rows = (level_ptr[level + 1] - p0) * nb;
        const float *xs = xstage + (size_t)(level & 1) * p.x_floats;
        for (int r_base = 0; r_base < rows; r_base += kTile) {
            // this lane finishes rows g and g + 8 of the tile, columns c0 and c0 + 1
            int rs[2], slot[2], e_at[2], e_end[2];
            bool live[2];
            size_t hrow[2];
            bool need_msg = false;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int r = r_base + g + 8 * i;
                live[i] = r < rows;
                const int q = live[i] ? (nb == 1 ? r : (int)__umulhi((unsigned)r, magic_nb)) : 0;
                rs[i] = live[i] ? r - q * nb : 0;
                const int4 m = meta[p0 + q];
                e_at[i] = m.x;
                e_end[i] = live[i] ? m.y : m.x;
                slot[i] = live[i] ? m.z : -1;
                hrow[i] = ((size_t)m.w * B + b_first + rs[i]) * D + c0;
                need_msg |= slot[i] >= 0;
            }
            // gather: sums of the neighbours' messages, the two rows side by side
            float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            // four neighbours at a time so that the slot and message loads overlap
            while (e_at[0] + 4 <= e_end[0] || e_at[1] + 4 <= e_end[1]) {
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    if (e_at[i] + 4 <= e_end[i]) {
                        int sl[4];
                        float2 m[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) sl[k] = nbr_slot[e_at[i] + k];
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            m[k] = *reinterpret_cast<const float2 *>(msg + (sl[k] * S + rs[i]) * D + c0);
                        acc[i].x += (m[0].x + m[1].x) + (m[2].x + m[3].x);
                        acc[i].y += (m[0].y + m[1].y) + (m[2].y + m[3].y);
                        e_at[i] += 4;
                    }
            }
            while (e_at[0] < e_end[0] || e_at[1] < e_end[1]) {
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    if (e_at[i] < e_end[i]) {
                        const float2 m = *reinterpret_cast<const float2 *>(
                            msg + (nbr_slot[e_at[i]] * S + rs[i]) * D + c0);
                        acc[i].x += m.x;
                        acc[i].y += m.y;
                        ++e_at[i];
                    }
            }
#pragma unroll
            for (int i = 0; i < 2; ++i)
                store_split(bufA + (g + 8 * i) * P + c0, TAIL, acc[i].x, acc[i].y);
            need_msg = __any_sync(0xffffffffu, need_msg);   // every warp sees all 16 rows
            group_sync();
            float c[4];
            tile_product<NKD>(wg1, bufA, P, lane, c);
            store_split(bufB + g * P + c0, TAIL, fmaxf(c[0] + bg1.x, 0.f), fmaxf(c[1] + bg1.y, 0.f));
            store_split(bufB + (g + 8) * P + c0, TAIL, fmaxf(c[2] + bg1.x, 0.f), fmaxf(c[3] + bg1.y, 0.f));
            group_sync();
            tile_product<NKD>(wg2, bufB, P, lane, c);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const float2 h = make_float2(fmaxf(c[2 * i] + bg2.x, 0.f), fmaxf(c[2 * i + 1] + bg2.y, 0.f));
                if (live[i]) *reinterpret_cast<float2 *>(H + hrow[i]) = h;
                store_split(bufA + (g + 8 * i) * P + c0, TAIL, h.x, h.y);
            }
            if (need_msg) {                                  // group-uniform
                // raw features (and zero padding) behind the d embedding columns
                for (int i = gt; i < kTile * (KF - D); i += GT) {
                    const int rr = i / (KF - D), k = i - rr * (KF - D);
                    const int r = r_base + rr;
                    const float v = (r < rows && k < F) ? xs[r * F + k] : 0.f;
                    const unsigned hv = tf32_round(v);
                    bufA[rr * P + D + k] = __uint_as_float(hv);
                    bufA[TAIL + rr * P + D + k] = __uint_as_float(tf32_round(v - __uint_as_float(hv)));
                }
                group_sync();
                tile_product<NKF>(wf1, bufA, P, lane, c);
                store_split(bufB + g * P + c0, TAIL, fmaxf(c[0] + bf1.x, 0.f), fmaxf(c[1] + bf1.y, 0.f));
                store_split(bufB + (g + 8) * P + c0, TAIL, fmaxf(c[2] + bf1.x, 0.f), fmaxf(c[3] + bf1.y, 0.f));
                group_sync();
                tile_product<NKD>(wf2, bufB, P, lane, c);
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    if (slot[i] >= 0)
                        *reinterpret_cast<float2 *>(msg + (slot[i] * S + rs[i]) * D + c0) =
                            make_float2(fmaxf(c[2 * i] + bf2.x, 0.f), fmaxf(c[2 * i + 1] + bf2.y, 0.f));
            }
            group_sync();     // tile buffers and message slots settled before the next tile
        }
        __pipeline_wait_prior(0);
        group_sync();
    }
}

template <int D>
bool relu2(const DevMlp &m, int in) {
    return m.n_layers == 2 && m.in_dim == in && m.hidden_dim == D && m.out_dim == D && m.act == 0 &&
           m.final_act == 1;
}

template <int D, int NKF>
cudaError_t launch(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap) {
    constexpr int P = 8 * NKF + 4;
    MmaPlan p;
    const int dirs_per_block = D == 32 ? 2 : 1;
    const int blocks_wanted = D == 32 ? di.sm_count : di.sm_count / 2;     // per direction set
    const int want = std::max(1, std::min(a.B, blocks_wanted));
    p.S = (a.B + want - 1) / want;
    // slices of 1, 2, 4, 8, 16, 32, ... states pack into 16-row tiles with less waste
    int pow2 = 1;
    while (pow2 < p.S) pow2 *= 2;
    p.S = std::min(pow2, a.B);
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    for (int dir = 0; dir < 2; ++dir) {
        const DevLevels &lv = a.lv[dir];
        p.int_floats[dir] = 4 * a.n + ((lv.n_levels + 1 + 3) & ~3) + ((lv.n_nbr + 3) & ~3);
    }
    auto x_floats = [&](int S) { return (a.max_level_width * S * a.F + 3) & ~3; };
    auto need = [&](int S) {
        size_t per_dir[2];
        for (int dir = 0; dir < 2; ++dir)
            per_dir[dir] = (size_t)p.int_floats[dir] + (size_t)a.lv[dir].n_slots * S * D +
                           2 * (size_t)x_floats(S) + 4 * (size_t)kTile * P;
        const size_t floats = dirs_per_block == 2 ? per_dir[0] + per_dir[1] : std::max(per_dir[0], per_dir[1]);
        return floats * sizeof(float);
    };
    while (p.S > 1 && need(p.S) > budget) --p.S;
    if (need(p.S) > budget) return cudaErrorNotSupported;
    // more slices than one wave of blocks: spread the batch evenly over the waves it takes
    {
        const int waves = ((a.B + p.S - 1) / p.S + want - 1) / want;
        p.S = std::min(p.S, (a.B + want * waves - 1) / (want * waves));
    }
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.x_floats = x_floats(p.S);
    p.smem_bytes = need(p.S);
    auto kern = embed_mma_kernel<D, NKF>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    err = launch_overlapped(overlap, kern, dim3(p.n_slices, D == 32 ? 1 : 2), dim3(256), p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace

bool embed_mma_applicable(const EmbedArgs &a) {
    if (a.F < 1 || a.F > 16) return false;
    for (int dir = 0; dir < 2; ++dir) {
        if (a.d == 32 && (!relu2<32>(a.f[dir], 32 + a.F) || !relu2<32>(a.g[dir], 32))) return false;
        if (a.d == 64 && (!relu2<64>(a.f[dir], 64 + a.F) || !relu2<64>(a.g[dir], 64))) return false;
    }
    return a.d == 32 || a.d == 64;
}

// Measured on B200: the tile kernel wins at d = 64 (1.3x over the FMA kernel on
// the NASNet-shaped workload) and loses at d = 32, where levels hold fewer rows
// than one 16-row tile and the long MMA latency sits on the level-to-level path.
bool embed_mma_preferred(const EmbedArgs &a) { return embed_mma_applicable(a) && a.d == 64; }

cudaError_t launch_embed_mma(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream,
                             bool overlap) {
    const int f8 = (a.F + 7) / 8;      // 1 or 2
    if (a.d == 32) return f8 == 1 ? launch<32, 5>(a, di, stream, overlap) : launch<32, 6>(a, di, stream, overlap);
    if (a.d == 64) return f8 == 1 ? launch<64, 9>(a, di, stream, overlap) : launch<64, 10>(a, di, stream, overlap);
    return cudaErrorNotSupported;
}

}  // namespace placeto
