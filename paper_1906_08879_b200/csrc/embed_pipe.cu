// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper) for d = 64 with
// two-layer ReLU networks of hidden width d, as a pipeline of layers:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]).
//
// A block owns a slice of the state batch and one direction and walks the
// levels of the graph; a level's rows (node, state) are cut into tiles of eight.
// Every layer of g and f has its own group of four warps, and a tile travels
// gather -> g layer 1 -> g layer 2 -> f layer 1 -> f layer 2 through rings of
// shared-memory buffers, handed over with named barriers (the producing group
// arrives, the consuming group waits in hardware). Several tiles of a level
// are in flight at once, one per layer, so the tensor pipes stay busy although
// each layer of one tile depends on the one before.
//
// Arithmetic: the product is computed transposed on mma.sync.m16n8k8 (TF32
// inputs, FP32 accumulate): the instruction's 16 rows are 16 output columns of
// the layer, its 8 columns the tile's rows. The weights (16 columns of one
// matrix per warp, split into a TF32 head and a TF32 tail) stay in registers as
// A fragments for the whole launch; the activations, split the same way by the
// warp that produced them, are B fragments read with ldmatrix (four warps read
// a tile instead of eight, and eight rows instead of sixteen padded ones).
// Three products are accumulated (head*head + head*tail + tail*head); the
// dropped tail*tail term is below 2^-22 relative.
//
// The warps of the last layer also gather: after the last tile of a level
// they sum the neighbours' messages for the first tiles of the next level (the
// messages live in shared-memory slots assigned on the host; a slot is never
// rewritten inside the level that still reads it). The raw features of the next
// level arrive by cp.async while the current level computes.
//
// There is no spin-wait in the kernel: every wait is a hardware barrier whose
// arrivals follow the data flow (gather -> layers), and the way back needs none
// because the group that takes tiles out at the end is the one that lets them in.
// Summation order is fixed: results are reproducible bit for bit.
#include <cuda_pipeline.h>

#include <algorithm>
#include <type_traits>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 64;
constexpr int kTile = 8;                 // rows of a tile
constexpr int kRing = 3;                 // tiles a buffer ring holds, and tiles in flight at most
constexpr int kStages = 4;               // g layer 1, g layer 2, f layer 1, f layer 2
constexpr int kGroupWarps = 4, kGroupThreads = 32 * kGroupWarps;
constexpr int kThreads = kStages * kGroupThreads;
constexpr int kP = kD + 4;               // row stride of a 64-wide tile and of a message (floats)
constexpr int kTail = kTile * kP;        // the tails of a tile follow its heads
constexpr int kFirstBar = 2;             // named barriers: 0 the block's, 1 the last layer's group, then ring x slot
constexpr int NKD = kD / 8;

struct PipePlan {
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
// round to nearest (ties away from zero) to TF32 with two integer operations
__device__ __forceinline__ float tf32_round(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    // volatile: the three accumulator chains have to stay interleaved as written (grouped by
    // accumulator, every instruction would wait the full 21 cycles for the one before)
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four 8 x 4 blocks of 32-bit words: lane i gives the address of row i % 8 of block i / 8 and
// receives, from block j, word lane % 4 of row lane / 4 -- the B fragments of two k-steps.
// `addr` is a shared-memory address, OFF a byte offset known at compile time (no address
// arithmetic per instruction).
template <int OFF>
__device__ __forceinline__ void ldmatrix4(unsigned (&r)[4], unsigned addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4+%5];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr), "n"(OFF)
                 : "memory");
}
template <int OFF>
__device__ __forceinline__ void ldmatrix2(unsigned (&r)[2], unsigned addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2+%3];"
                 : "=r"(r[0]), "=r"(r[1])
                 : "r"(addr), "n"(OFF)
                 : "memory");
}
// One warp's 16 columns [c0, c0 + 16) of a K x d matrix as A fragments of the transposed
// product, heads and tails: for k-step ks, with g = lane / 4 and t = lane % 4,
//   a0 = W[8 ks + t][c0 + g], a1 = W[8 ks + t][c0 + g + 8], a2, a3 = the same at k + 4.
template <int NKS>
struct AFrag {
    unsigned h[NKS][4], l[NKS][4];
    __device__ __forceinline__ void load(const float *W, int ld, int n_rows, int c0, int lane) {
        const int g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int ks = 0; ks < NKS; ++ks)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = 8 * ks + t + 4 * (i >> 1), c = c0 + g + 8 * (i & 1);
                const float w = k < n_rows ? W[(size_t)k * ld + c] : 0.f;
                h[ks][i] = tf32_of(w);
                l[ks][i] = tf32_of(w - __uint_as_float(h[ks][i]));
            }
    }
};

// c = (this warp's 16 columns of W)^T x (tile)^T for a tile of 8 rows in shared memory, in the
// C-fragment layout
//   c[0], c[1] = (column g,     rows 2t, 2t + 1);  c[2], c[3] = (column g + 8, same rows),
// plus the bias of the two columns (the accumulators start from it).
// `heads` is this lane's ldmatrix address in the tile's heads (row lane % 8, block lane / 8, see
// ldmatrix_lane_offset), `tails` the same in its tails. NKS k-steps: d / 8 for the embedding
// columns, one or two more for the raw features behind them (f's first layer). Three independent
// accumulators: a dependent mma.sync can issue after about 21 cycles and the pipe takes one from
// a warp every 8, so three chains keep it fed. The fragments of the next pair of k-steps are
// requested before the products of this one.
__device__ __forceinline__ int ldmatrix_lane_offset(int lane, int P) {
    return ((lane & 7) * P + 4 * (lane >> 3)) * (int)sizeof(float);
}
template <int NKS>
__device__ __forceinline__ void tile_product(const AFrag<NKS> &w, unsigned heads, unsigned tails, float b_lo, float b_hi,
                                             float (&c)[4]) {
    static_assert(NKD == 8 && NKS >= NKD && NKS <= NKD + 2, "four pairs of k-steps written out below, and a tail");
    float hh[4] = {b_lo, b_lo, b_hi, b_hi}, hl[4] = {0.f, 0.f, 0.f, 0.f}, lh[4] = {0.f, 0.f, 0.f, 0.f};     // bias: columns g, g + 8
    auto pair = [&](int kp, const unsigned (&bh)[4], const unsigned (&bl)[4], int count) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (j >= count) break;
            const int ks = 2 * kp + j;
            mma_tf32(lh, w.l[ks], bh[2 * j], bh[2 * j + 1]);
            mma_tf32(hl, w.h[ks], bl[2 * j], bl[2 * j + 1]);
            mma_tf32(hh, w.h[ks], bh[2 * j], bh[2 * j + 1]);
        }
    };
    unsigned bh0[4], bl0[4], bh1[4], bl1[4];
    ldmatrix4<0>(bh0, heads);
    ldmatrix4<0>(bl0, tails);
    ldmatrix4<64>(bh1, heads);
    ldmatrix4<64>(bl1, tails);
    pair(0, bh0, bl0, 2);
    ldmatrix4<128>(bh0, heads);
    ldmatrix4<128>(bl0, tails);
    pair(1, bh1, bl1, 2);
    ldmatrix4<192>(bh1, heads);
    ldmatrix4<192>(bl1, tails);
    pair(2, bh0, bl0, 2);
    if (NKS == NKD + 2) {
        ldmatrix4<256>(bh0, heads);
        ldmatrix4<256>(bl0, tails);
    } else if (NKS == NKD + 1) {
        unsigned eh[2], el[2];      // lanes 0 .. 15 give the addresses: blocks 0 and 1, as above
        ldmatrix2<256>(eh, heads);
        ldmatrix2<256>(el, tails);
        bh0[0] = eh[0]; bh0[1] = eh[1];
        bl0[0] = el[0]; bl0[1] = el[1];
    }
    pair(3, bh1, bl1, 2);
    if (NKS > NKD) pair(4, bh0, bl0, NKS - NKD);
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = hh[i] + (hl[i] + lh[i]);
}

// head and tail of one activation into a tile
__device__ __forceinline__ void store_split(float *head, int tail, float x) {
    const float hx = tf32_round(x);
    head[0] = hx;
    head[tail] = tf32_round(x - hx);
}

// Named barrier `id`: the 128 threads of the producing group announce a tile (without
// waiting), the 128 of the consuming group wait for it. The fence makes the producer's
// shared-memory writes visible before the arrival counts.
__device__ __forceinline__ void tile_ready(int id) {
    __threadfence_block();
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "n"(2 * kGroupThreads) : "memory");
}
__device__ __forceinline__ void await_tile(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(2 * kGroupThreads) : "memory");
}

template <int NKF>   // k-steps of f's first layer, 8 NKF >= d + F
__global__ void __launch_bounds__(kThreads, 1)
embed_pipe_kernel(const EmbedArgs a, const PipePlan p) {
    static_assert(NKF == NKD + 1 || NKF == NKD + 2, "raw features take one or two k-steps");
    constexpr int KF = 8 * NKF;
    constexpr int PF = KF + 4;                       // row stride of the tiles that f's first layer reads
    constexpr int XC = KF - kD;                      // columns behind the embedding: raw features, zero padded
    static_assert(kTile * XC <= kGroupThreads, "one feature word per thread and tile");
    extern __shared__ __align__(16) float smem[];
    dependents_may_start();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stage = warp >> 2;                     // the layer this warp computes
    const int c0 = 16 * (warp & 3);                  // its block of output columns
    const int gt = threadIdx.x & (kGroupThreads - 1);
    const int g = lane >> 2, t = lane & 3;
    const int dir = (int)blockIdx.y;
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F, S = p.S;
    const int b_first = blockIdx.x * S;
    const int nb = min(S, B - b_first);

    // ---- shared memory: [schedule][message slots][x staging x2][four rings of tiles]
    // level_ptr, nbr_slot and one packed record per position:
    //   meta[p] = {first neighbour entry, end of neighbour entries, own slot, node id}
    int *ism = reinterpret_cast<int *>(smem);
    int4 *meta_w = reinterpret_cast<int4 *>(ism);
#pragma unroll 1
    for (int i = threadIdx.x; i < a.n; i += kThreads) {
        meta_w[i] = make_int4(lv.nbr_ptr[i], lv.nbr_ptr[i + 1], lv.own_slot[i], lv.order[i]);
        PLACETO_DEBUG_CHECK(a.status, lv.nbr_ptr[i] >= 0 && lv.nbr_ptr[i] <= lv.nbr_ptr[i + 1] &&
                                          lv.nbr_ptr[i + 1] <= lv.n_nbr && lv.own_slot[i] >= -1 &&
                                          lv.own_slot[i] < lv.n_slots && lv.order[i] >= 0 && lv.order[i] < a.n);
    }
#pragma unroll 1
    for (int e = threadIdx.x; e < lv.n_nbr; e += kThreads)
        PLACETO_DEBUG_CHECK(a.status, lv.nbr_slot[e] >= 0 && lv.nbr_slot[e] < lv.n_slots);
    PLACETO_DEBUG_CHECK(a.status, nb >= 1 && b_first + nb <= B);
    ism += 4 * a.n;
    auto stage_ints = [&](const int *src, int count) {
        int *dst = ism;
#pragma unroll 1
        for (int i = threadIdx.x; i < count; i += kThreads) dst[i] = src[i];
        ism += (count + 3) & ~3;
        return (const int *)dst;
    };
    const int4 *meta = meta_w;
    const int *level_ptr = stage_ints(lv.level_ptr, lv.n_levels + 1);
    const int *nbr_slot = stage_ints(lv.nbr_slot, lv.n_nbr);
    float *msg = smem + p.int_floats[dir];                      // [n_slots][S][kP]
    float *xstage = msg + (size_t)lv.n_slots * S * kP;          // [2][x_floats]
    float *ring0 = xstage + 2 * (size_t)p.x_floats;             // gather -> g layer 1
    float *ring1 = ring0 + kRing * 2 * kTail;                   // g layer 1 -> g layer 2
    float *ring2 = ring1 + kRing * 2 * kTail;                   // g layer 2 (+ raw features) -> f layer 1
    float *ring3 = ring2 + kRing * 2 * kTile * PF;              // f layer 1 -> f layer 2
    const float *X = a.X;
    float *__restrict__ H = a.H[dir];

    const int col = c0 + g;                          // this lane finishes columns col and col + 8 of rows 2t, 2t + 1
    // Hand-over: named barrier kFirstBar + ring * kRing + slot. There is no barrier for the way
    // back: the last layer's group, which also feeds the first ring, lets tile n + kRing in only
    // after it has taken tile n out of the last ring, so at most kRing tiles are between the
    // rings at any time and a slot is never rewritten before everybody has read it.

    // exact division of small non-negative numbers by a per-block constant
    const unsigned magic_nb = (unsigned)((0x100000000ull + nb - 1) / nb);
    auto node_of_row = [&](int r) { return nb == 1 ? r : (int)__umulhi((unsigned)r, magic_nb); };
    auto tiles_of = [&](int level) {
        return ((level_ptr[level + 1] - level_ptr[level]) * nb + kTile - 1) / kTile;
    };
    __syncthreads();              // schedule staged
    dependency_wait();            // the raw features may come from a kernel that is still running

    int slot = 0;                 // ring slot of the tile this warp takes next (tiles taken so far modulo kRing)
    int g_slot = 0;               // last layer: ring slot of the tile gathered next
    int g_level = 0, g_j = 0;     //             the next tile to gather

    // Last layer: sum of the neighbours' messages of tile j of a level, split, into the first
    // ring: thread (row gt / 16, columns 4 (gt % 16) ...) of the group.
    auto gather = [&](int level, int j) {
        const int p0 = level_ptr[level], rows = (level_ptr[level + 1] - p0) * nb;
        const int rr = gt >> 4, c4 = 4 * (gt & 15);
        const int r = kTile * j + rr;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < rows) {
            const int q = node_of_row(r), s = r - q * nb;
            const int4 m = meta[p0 + q];
            const float *from = msg + s * kP + c4;
#pragma unroll 2
            for (int e = m.x; e < m.y; ++e) {
                const float4 v = *reinterpret_cast<const float4 *>(from + (size_t)nbr_slot[e] * S * kP);
                acc.x += v.x;
                acc.y += v.y;
                acc.z += v.z;
                acc.w += v.w;
            }
        }
        float *out = ring0 + g_slot * 2 * kTail + rr * kP + c4;
        const float4 head = make_float4(tf32_round(acc.x), tf32_round(acc.y), tf32_round(acc.z), tf32_round(acc.w));
        *reinterpret_cast<float4 *>(out) = head;
        *reinterpret_cast<float4 *>(out + kTail) =
            make_float4(tf32_round(acc.x - head.x), tf32_round(acc.y - head.y), tf32_round(acc.z - head.z),
                        tf32_round(acc.w - head.w));
        tile_ready(kFirstBar + g_slot);
        g_slot = g_slot == kRing - 1 ? 0 : g_slot + 1;
    };
    // First layer of g: the raw features of a level, one level ahead. Every thread fetches exactly
    // the word it will itself copy into each tile, so its own wait is all the synchronisation needed.
    const int x_row = gt / XC, x_col = gt - x_row * XC;          // gt < kTile * XC: a word of every tile
    const bool x_mine = gt < kTile * XC;
    auto prefetch = [&](int level) {
        const int p0 = level_ptr[level], rows = (level_ptr[level + 1] - p0) * nb;
        float *dst = xstage + (size_t)(level & 1) * p.x_floats;
        if (x_mine && x_col < F) {
#pragma unroll 1
            for (int r = x_row; r < rows; r += kTile) {
                const int q = node_of_row(r);
                __pipeline_memcpy_async(dst + r * F + x_col,
                                        X + ((size_t)meta[p0 + q].w * B + b_first + (r - q * nb)) * F + x_col, 4);
            }
        }
        __pipeline_commit();
    };

    // One copy of the walk per layer, so that what differs between the layers (which ring, the
    // raw-feature columns, where h_v and m_u go, the gather) is decided at compile time.
    auto walk = [&](auto stage_constant) {
    constexpr int STAGE = decltype(stage_constant)::value;
    constexpr bool second = STAGE & 1;
    constexpr bool wide = STAGE == 2;                // f's first layer also reads the raw features
    constexpr int NKW = wide ? NKF : NKD;
    const DevMlp net = STAGE < 2 ? a.g[dir] : a.f[dir];
    AFrag<NKW> w;
    w.load(second ? net.W2 : net.W1, kD, wide ? kD + F : kD, c0, lane);
    const float b_lo = (second ? net.b2 : net.b1)[col], b_hi = (second ? net.b2 : net.b1)[col + 8];
    const float *in_ring = STAGE == 0 ? ring0 : STAGE == 1 ? ring1 : STAGE == 2 ? ring2 : ring3;
    float *out_ring = STAGE == 0 ? ring1 : STAGE == 1 ? ring2 : ring3;
    constexpr int in_P = STAGE == 2 ? PF : kP, out_P = STAGE == 1 ? PF : kP;
    constexpr int in_bar = kFirstBar + STAGE * kRing, out_bar = in_bar + kRing;
    // this lane's ldmatrix address in slot 0 of the input ring, and the bytes of a tile (heads + tails)
    const unsigned in_lane = smem_addr(in_ring) + ldmatrix_lane_offset(lane, in_P);
    constexpr unsigned in_tile_bytes = 2 * kTile * in_P * sizeof(float);
    // The walk starts one level early, with nothing to compute: the last layer's group gathers
    // the first tiles of level 0 there and the first layer of g requests its raw features, in
    // the same code that does it between two levels (one call site each, inlined).
#pragma unroll 1
    for (int level = -1; level < lv.n_levels; ++level) {
        const int p0 = level < 0 ? 0 : level_ptr[level], rows = level < 0 ? 0 : (level_ptr[level + 1] - p0) * nb;
        const int n_tiles = level < 0 ? (STAGE == 3 ? 1 : 0) : (rows + kTile - 1) / kTile;
        const float *xs = xstage + (size_t)(level & 1) * p.x_floats;
        if (STAGE == 0) __pipeline_wait_prior(0);          // this level's raw features: requested a level ago
#pragma unroll 1
        for (int j = 0; j < n_tiles; ++j) {
            if (level >= 0) {
                // ---- before the tile arrives: whatever does not depend on it
                float *dst[2] = {nullptr, nullptr};             // second layers: where rows 2t, 2t + 1 go (h_v / m_u)
                if (second) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int r = kTile * j + 2 * t + i;
                        if (r < rows) {
                            const int q = node_of_row(r);
                            const int4 m = meta[p0 + q];
                            if (STAGE == 1) dst[i] = H + ((size_t)m.w * B + b_first + (r - q * nb)) * kD + col;
                            else if (m.z >= 0) dst[i] = msg + ((size_t)m.z * S + (r - q * nb)) * kP + col;
                        }
                    }
                }
                if (STAGE == 0 && x_mine) {
                    // The raw features (zero padded) behind the d embedding columns of the tile that f's
                    // first layer will read, two rings on: its slot is free (at most kRing tiles are
                    // in flight), and this group has the lightest layer.
                    const int r = kTile * j + x_row;
                    store_split(ring2 + slot * 2 * kTile * PF + x_row * PF + kD + x_col, kTile * PF,
                                (r < rows && x_col < F) ? xs[r * F + x_col] : 0.f);
                }
                await_tile(in_bar + slot);
                float c[4];
                const unsigned heads = in_lane + slot * in_tile_bytes;
                tile_product<NKW>(w, heads, heads + in_tile_bytes / 2, b_lo, b_hi, c);
                // (row 2t, col), (2t + 1, col), (2t, col + 8), (2t + 1, col + 8)
                const float v[4] = {fmaxf(c[0], 0.f), fmaxf(c[1], 0.f), fmaxf(c[2], 0.f), fmaxf(c[3], 0.f)};
                if (STAGE != 3) {
                    float *out = out_ring + slot * 2 * kTile * out_P + 2 * t * out_P + col;
                    const int tail = kTile * out_P;
                    store_split(out, tail, v[0]);
                    store_split(out + out_P, tail, v[1]);
                    store_split(out + 8, tail, v[2]);
                    store_split(out + out_P + 8, tail, v[3]);
                    tile_ready(out_bar + slot);
                }
                if (second) {
#pragma unroll
                    for (int i = 0; i < 2; ++i)
                        if (dst[i] != nullptr) {
                            dst[i][0] = v[i];
                            dst[i][8] = v[2 + i];
                        }
                }
                slot = slot == kRing - 1 ? 0 : slot + 1;
            }
            if (STAGE == 3) {
                // Sums for the tiles ahead. Inside a level: one more tile for the one just taken
                // (this level's messages go to slots that no row of this level reads). After the
                // level's last tile: all its messages are written (group barrier), and the first
                // tiles of the next level follow.
                const bool last = j == n_tiles - 1;
                int upto = min(n_tiles, j + 1 + kRing);
                if (last) {
                    asm volatile("bar.sync 1, %0;" ::"n"(kGroupThreads) : "memory");
                    g_level = level + 1;
                    g_j = 0;
                    upto = level + 1 < lv.n_levels ? min(kRing, tiles_of(level + 1)) : 0;
                }
#pragma unroll 1
                for (; g_j < upto; ++g_j) gather(g_level, g_j);
            }
        }
        if (STAGE == 0 && level + 1 < lv.n_levels) prefetch(level + 1);      // the other buffer: its level is done
    }
    };
    switch (stage) {
        case 0: walk(std::integral_constant<int, 0>{}); break;
        case 1: walk(std::integral_constant<int, 1>{}); break;
        case 2: walk(std::integral_constant<int, 2>{}); break;
        default: walk(std::integral_constant<int, 3>{}); break;
    }
}

bool relu2(const DevMlp &m, int in) {
    return m.n_layers == 2 && m.in_dim == in && m.hidden_dim == kD && m.out_dim == kD && m.act == 0 &&
           m.final_act == 1;
}

template <int NKF>
cudaError_t launch(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap) {
    constexpr int PF = 8 * NKF + 4;
    PipePlan p;
    // one block per SM at most: half the SMs per direction
    const int want = std::max(1, std::min(a.B, di.sm_count / 2));
    p.S = (a.B + want - 1) / want;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    for (int dir = 0; dir < 2; ++dir) {
        const DevLevels &lv = a.lv[dir];
        p.int_floats[dir] = 4 * a.n + ((lv.n_levels + 1 + 3) & ~3) + ((lv.n_nbr + 3) & ~3);
    }
    auto x_floats = [&](int S) { return (a.max_level_width * S * a.F + 3) & ~3; };
    auto need = [&](int S) {
        size_t worst = 0;
        for (int dir = 0; dir < 2; ++dir)
            worst = std::max(worst, (size_t)p.int_floats[dir] + (size_t)a.lv[dir].n_slots * S * kP);
        const size_t floats = worst + 2 * (size_t)x_floats(S) + 3 * (size_t)kRing * 2 * kTail +
                              (size_t)kRing * 2 * kTile * PF;
        return floats * sizeof(float);
    };
    while (p.S > 1 && need(p.S) > budget) --p.S;
    if (need(p.S) > budget) return cudaErrorNotSupported;
    // Shared memory may force more slices than one wave of blocks holds: spread the batch evenly over
    // the waves it then takes (two full waves finish before one full wave and a ragged one of larger slices)
    const int waves = ((a.B + p.S - 1) / p.S + want - 1) / want;
    p.S = std::min(p.S, (a.B + want * waves - 1) / (want * waves));
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.x_floats = x_floats(p.S);
    p.smem_bytes = need(p.S);
    auto kern = embed_pipe_kernel<NKF>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    err = launch_overlapped(overlap, kern, dim3(p.n_slices, 2), dim3(kThreads), p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace

bool embed_pipe_applicable(const EmbedArgs &a) {
    if (a.d != kD || a.F < 1 || a.F > 16) return false;
    for (int dir = 0; dir < 2; ++dir)
        if (!relu2(a.f[dir], kD + a.F) || !relu2(a.g[dir], kD)) return false;
    return true;
}

// Measured on B200 on the NASNet-shaped graph (n = 2130, 744 levels), pipeline against the
// 16-row-tile kernel, ms: 0.90 / 1.72 at B = 64, 1.37 / 2.09 at 256, 2.10 / 2.94 at 512, 3.75 / 4.92 at
// 1024, 7.48 / 9.19 at 2048, 14.9 / 18.2 at 4096: the pipeline is taken wherever it applies.
bool embed_pipe_preferred(const EmbedArgs &a, const DeviceInfo &) { return embed_pipe_applicable(a); }

cudaError_t launch_embed_pipe(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap) {
    return a.F <= 8 ? launch<9>(a, di, stream, overlap) : launch<10>(a, di, stream, overlap);
}

}  // namespace placeto
