// Step 2 of the policy (Sec. 2.2 step 2 of the Placeto paper) for d = 64 on the
// fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_u = f([h_u || x_u]),
// f and g two-layer ReLU networks of hidden width 64.
//
// Schedule. As in the other sweep kernels a block owns one direction and a
// slice of S states and walks all levels on its own (states never interact), the
// messages live in shared-memory slots assigned on the host. A level's rows
// (node, state) of the block form one tile of R <= 64 rows (wider levels take
// several tiles), and every layer of the tile is ONE accumulation chain of eight
// tensor-core instructions.
//
// Arithmetic. FP32 accuracy on TF32 operands: every value is split into a TF32
// head and tail. The layer is computed transposed, out^T = W^T act^T, so that
// the instruction's M dimension carries the 64 output columns twice (rows of
// W^T's head and of its tail stacked: M = 128) and its N dimension the tile's
// rows twice (heads in columns [0, R8), tails in [R8, 2 R8), R8 = R rounded up
// to 8). One instruction per 8-wide k-step then yields all four partial
// products head*head, head*tail, tail*head, tail*tail in the 128 x 2 R8
// accumulator, and the layer costs 8 instructions whatever R is (an
// instruction's cost is flat up to N of about 96).
//
// Roles. Sixteen epilogue warps own the accumulator: warp w reads the 32 lanes
// of quadrant w % 4 (16 output columns: lanes j and j + 16 hold the head and
// tail rows of column 16 (w % 4) + j) for the 8-row units u = w / 4 (mod 4), adds
// the four partial products (one shuffle between the lane halves), applies bias
// and ReLU, splits the result and stores it as the next layer's operand. The
// raw-feature part of f's first layer (F <= 16 columns) is a short FP32 FMA loop
// done by the same threads while the tensor cores run. One thread of a control
// warp issues the instructions; a loader warp stages the schedule records and
// raw features two levels ahead. All hand-offs are mbarriers with bounded
// waits: a wait that runs out raises a flag, every role leaves its loop, the
// tensor memory is released and the status word reports the time-out.
#include <algorithm>
#include <cstdio>
#include <type_traits>

#include "kernels.cuh"

namespace placeto {

namespace {

// Build with -DPLACETO_PHASE_TIMERS to have block (0, 0) print, per role, the cycles it spent
// in each phase of a level (sums over all levels, from clock64()).
#ifdef PLACETO_PHASE_TIMERS
#define PT_DECL(n) long long pt_[n] = {}; long long pt_last_ = clock64()
#define PT(i) do { const long long pt_now_ = clock64(); pt_[i] += pt_now_ - pt_last_; pt_last_ = pt_now_; } while (0)
#else
#define PT_DECL(n) do { } while (0)
#define PT(i) do { } while (0)
#endif

constexpr int D = 64;
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kEpiThreads + 64;      // + control warp + loader warp
constexpr int kCtlWarp = kEpiWarps;            // the warp after it loads
constexpr int kTileRows = 64;                   // rows of a tile (R8 <= 64, N <= 128)
constexpr int kTmemCols = 128;
constexpr int kRing = 3;                        // staged levels in flight
constexpr int LBO_A = 128;                      // weights: the 16-byte k-chunks of 8 rows, contiguous
constexpr int A_BYTES = 128 * D * 4;            // one stacked matrix: 128 rows x 64 k
constexpr int LBO_B = 144;                      // activations: 16 B of padding per k-chunk, so that a warp's
                                                // column-wise 4-byte stores fall into 32 different banks
constexpr int SBO_B = (D / 4) * LBO_B;          // 2304 B per group of 8 rows
constexpr int B_BYTES = (2 * kTileRows / 8) * SBO_B;

struct TcPlan {
    int S, n_slices;
    int off_msg, off_ring, ring_bytes, off_rec, off_nslot, off_x;   // byte offsets (ring-relative for the last three)
    int smem_bytes;
};

__device__ __forceinline__ uint32_t a_off(int i, int k) {
    return (uint32_t)((i >> 3) * (D * 32) + (k >> 2) * LBO_A + (i & 7) * 16 + (k & 3) * 4);
}
// Shared-memory matrix descriptor, no swizzle, K-major: 8 x 16-byte core matrices,
// `lbo` bytes between core matrices along k, `sbo` bytes between groups of 8 rows.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
// Instruction descriptor: FP32 accumulate, TF32 A and B, both K-major, M x N.
__device__ __forceinline__ uint32_t make_idesc(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accum) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Bounded wait for phase `parity`; gives up early when another thread has raised *abort.
// Two forms. Suspending (long waits: the loader's, a level's staged data): each try parks the
// thread in hardware for up to about a millisecond, so it takes no issue slots from the working
// warps; 256 tries bound the wait to a fraction of a second. Polling (the hand-offs on the
// critical path, where the wake-up latency of a parked thread would show): a bounded spin.
template <bool kSuspend>
__device__ __forceinline__ bool wait_or_abort(unsigned long long *bar, unsigned parity, volatile int *abort) {
    if (kSuspend) {
        for (int i = 0; i < 256; ++i) {
            unsigned done;
            asm volatile(
                "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
                : "=r"(done)
                : "r"(smem_addr(bar)), "r"(parity), "r"(1000000u)
                : "memory");
            if (done) return true;
            if (*abort) return false;
        }
    } else {
        for (int i = 0; i < (1 << 22); ++i) {
            unsigned done;
            asm volatile(
                "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                : "=r"(done)
                : "r"(smem_addr(bar)), "r"(parity)
                : "memory");
            if (done) return true;
            if ((i & 63) == 63 && *abort) return false;
        }
    }
    *abort = 1;
    return false;
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
// orders this thread's shared-memory stores before the tensor core's reads of them
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Two 8-column loads from this warp's 32 lanes of tensor memory, and the wait for both.
__device__ __forceinline__ void tmem_ld8x2(uint32_t ta, uint32_t tb, uint32_t (&a)[8], uint32_t (&b)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%16];\n"
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%8,%9,%10,%11,%12,%13,%14,%15}, [%17];\n"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]), "=r"(a[6]), "=r"(a[7]),
          "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]), "=r"(b[6]), "=r"(b[7])
        : "r"(ta), "r"(tb)
        : "memory");
}

__device__ __forceinline__ unsigned tf32_round(float x) { return (__float_as_uint(x) + 0x1000u) & 0xffffe000u; }

// Rows 8u .. 8u + 7 of a layer's output for this thread's column. Lanes below 16
// (head rows of the weights) hold head*head + head*tail after the first add, the
// others tail*head + tail*tail; the halves swap four rows each, so that lanes
// below 16 finish rows 8u + i and the others rows 8u + 4 + i (i = 0 .. 3).
__device__ __forceinline__ void load_unit(uint32_t tmem_q, int u, int R8, bool lo, float (&v)[4]) {
    uint32_t a[8], b[8];
    tmem_ld8x2(tmem_q + 8 * u, tmem_q + R8 + 8 * u, a, b);
    float p[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) p[i] = __uint_as_float(a[i]) + __uint_as_float(b[i]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float send = lo ? p[4 + i] : p[i];
        const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
        v[i] = (lo ? p[i] : p[4 + i]) + recv;
    }
}

// operand element (row, k): head at row, tail at R8 + row; `at` = bufB + b_off(row, k)
__device__ __forceinline__ void store_act(unsigned char *at, int tail_bytes, float x) {
    const unsigned h = tf32_round(x);
    const float hf = __uint_as_float(h);
    *reinterpret_cast<float *>(at) = hf;
    *reinterpret_cast<float *>(at + tail_bytes) = __uint_as_float(tf32_round(x - hf));
}

// W [64 rows of k][64] row-major (global) -> stacked operand: row 32q + j = head of
// column 16q + j, row 32q + 16 + j = its tail.
__device__ __forceinline__ void build_a_stack(unsigned char *dst, const float *W, int tid, int nthreads) {
    for (int idx = tid; idx < 128 * D; idx += nthreads) {
        const int k = idx >> 7, i = idx & 127;
        const int c = 16 * (i >> 5) + (i & 15), part = (i >> 4) & 1;
        const float w = W[k * D + c];
        const unsigned h = tf32_round(w);
        *reinterpret_cast<unsigned *>(dst + a_off(i, k)) = part ? tf32_round(w - __uint_as_float(h)) : h;
    }
}

__global__ void __launch_bounds__(kThreads, 1) embed_tc_kernel(const EmbedArgs a, const TcPlan p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ unsigned long long bar_mma, bar_epi, bar_level, bar_drain;
    __shared__ unsigned long long bar_meta[kRing], bar_free[kRing];
    __shared__ uint32_t tmem_s;
    __shared__ int abort_s;
    dependents_may_start();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int dir = blockIdx.y;
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F, S = p.S;
    const int b_first = blockIdx.x * S;
    const int nb = min(S, B - b_first);
    const int n_levels = lv.n_levels;

    unsigned char *sA = smem;                                  // g1, g2, f1 (embedding part), f2
    unsigned char *sB = smem + 4 * A_BYTES;
    float *msg = reinterpret_cast<float *>(smem + p.off_msg);  // [n_slots][S][64]
    unsigned char *ring = smem + p.off_ring;
    // one staged level: {width, rows} | a record per row | neighbour slots | raw features
    auto ring_head = [&](int slot) { return reinterpret_cast<int *>(ring + slot * p.ring_bytes); };
    auto ring_rec = [&](int slot) { return reinterpret_cast<int4 *>(ring + slot * p.ring_bytes + p.off_rec); };
    auto ring_nslot = [&](int slot) { return reinterpret_cast<int *>(ring + slot * p.ring_bytes + p.off_nslot); };
    auto ring_x = [&](int slot) { return reinterpret_cast<float *>(ring + slot * p.ring_bytes + p.off_x); };

    if (warp == kCtlWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_s)),
                     "n"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(&bar_mma, 1);
        mbar_init(&bar_epi, kEpiThreads);
        mbar_init(&bar_level, kEpiThreads);
        mbar_init(&bar_drain, 1);
        for (int i = 0; i < kRing; ++i) {
            mbar_init(&bar_meta[i], 32);
            mbar_init(&bar_free[i], kEpiThreads);
        }
        abort_s = 0;
    }
    const DevMlp f = a.f[dir], gm = a.g[dir];
    for (int i = tid; i < B_BYTES / 4; i += kThreads) reinterpret_cast<float *>(sB)[i] = 0.f;
    build_a_stack(sA + 0 * A_BYTES, gm.W1, tid, kThreads);
    build_a_stack(sA + 1 * A_BYTES, gm.W2, tid, kThreads);
    build_a_stack(sA + 2 * A_BYTES, f.W1, tid, kThreads);      // rows 0 .. 63: the embedding part of [h || x]
    build_a_stack(sA + 3 * A_BYTES, f.W2, tid, kThreads);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_s;
    volatile int *abort = &abort_s;
    dependency_wait();          // the raw features may come from a kernel that is still running

    if (warp < kEpiWarps) {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp & 3, uu = warp >> 2;
        const bool lo = lane < 16;
        const int c = 16 * q + (lane & 15), r_add = lo ? 0 : 4;
        const uint32_t tmem_q = tmem + ((uint32_t)(32 * q) << 16);
        const float bg1 = gm.b1[c], bg2 = gm.b2[c], bf1 = f.b1[c], bf2 = f.b2[c];
        float w1x[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) w1x[k] = k < F ? f.W1[(D + k) * D + c] : 0.f;
        float *__restrict__ H = a.H[dir];
        const int SD = S * D;
        unsigned char *col_base = sB + (c >> 2) * LBO_B + (c & 3) * 4 + r_add * 16;   // + unit * SBO_B + i * 16
        const int4 *rec = nullptr;
        const int *nslot = nullptr;
        const float *xs = nullptr;
        unsigned k_mma = 0;
        // One tile (R <= 32 nu rows) through gather and the four layers; false after a time-out.
        // Per row the loader left {first neighbour entry | entries << 16, state, own message
        // offset or -1, row of H}.
        auto epilogue_tile = [&](auto nu, int r_base, int R) -> bool {
            const int R8 = (R + 7) & ~7, units = R8 >> 3;
            const int tail_bytes = units * SBO_B;
                int hrow[decltype(nu)::value][4], mown[decltype(nu)::value][4];
            float xp[decltype(nu)::value][4], hv[decltype(nu)::value][4];  // raw-feature part of f's first layer; h
            // ---- gather: sums of the neighbours' messages -> operand of g's first layer
        #pragma unroll
            for (int j = 0; j < decltype(nu)::value; ++j) {
                const int u = uu + 4 * j;
                if (u < units) {
                    int4 rc[4];
                    float acc[4];
        #pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = 8 * u + i + r_add;
                        rc[i] = r < R ? rec[r_base + r] : make_int4(0, 0, -1, -1);
                    }
        #pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        hrow[j][i] = rc[i].w;
                        mown[j][i] = rc[i].z;
                        const int cnt = rc[i].x >> 16;
                        acc[i] = cnt > 0 ? msg[nslot[rc[i].x & 0xffff] * SD + rc[i].y * D + c] : 0.f;
                    }
        #pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int e0 = rc[i].x & 0xffff, cnt = rc[i].x >> 16;
                        for (int k = 1; k < cnt; ++k) acc[i] += msg[nslot[e0 + k] * SD + rc[i].y * D + c];
                        store_act(col_base + u * SBO_B + i * 16, tail_bytes, acc[i]);
                    }
                } else {
        #pragma unroll
                    for (int i = 0; i < 4; ++i) hrow[j][i] = mown[j][i] = -1;
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar_epi);
            // while the tensor cores run g's first layer: the raw-feature part of f's first layer
            // (F <= 16 columns) on the FMA pipes
        #pragma unroll
            for (int j = 0; j < decltype(nu)::value; ++j)
        #pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float s = bf1;
                    if (hrow[j][i] >= 0) {
                        const float *xr = xs + (size_t)(r_base + 8 * (uu + 4 * j) + i + r_add) * F;
                        if ((F & 3) == 0) {
        #pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                if (4 * k4 < F) {
                                    const float4 t = reinterpret_cast<const float4 *>(xr)[k4];
                                    s = fmaf(t.x, w1x[4 * k4], s);
                                    s = fmaf(t.y, w1x[4 * k4 + 1], s);
                                    s = fmaf(t.z, w1x[4 * k4 + 2], s);
                                    s = fmaf(t.w, w1x[4 * k4 + 3], s);
                                }
                        } else {
        #pragma unroll
                            for (int k = 0; k < 16; ++k)
                                if (k < F) s = fmaf(xr[k], w1x[k], s);
                        }
                    }
                    xp[j][i] = s;
                }
            // ---- the four layers: g1, g2 (h), f1, f2 (message)
        #pragma unroll 1
            for (int layer = 0; layer < 4; ++layer) {
                const bool ok = __all_sync(0xffffffffu, wait_or_abort<true>(&bar_mma, k_mma++ & 1, abort));
                if (!ok) return false;
                tc_fence_after();
                const float bias = layer == 0 ? bg1 : layer == 1 ? bg2 : bf2;
        #pragma unroll
                for (int j = 0; j < decltype(nu)::value; ++j) {
                    const int u = uu + 4 * j;
                    if (u < units) {
                        float v[4];
                        load_unit(tmem_q, u, R8, lo, v);
        #pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float val = fmaxf(v[i] + (layer == 2 ? xp[j][i] : bias), 0.f);
                            if (layer == 3) {
                                if (mown[j][i] >= 0) msg[mown[j][i] + c] = val;
                            } else {
                                store_act(col_base + u * SBO_B + i * 16, tail_bytes, val);
                            }
                            if (layer == 1) hv[j][i] = val;
                        }
                    }
                }
                if (layer < 3) {
                    fence_async_smem();
                    tc_fence_before();
                    mbar_arrive(&bar_epi);
                } else {
                    tc_fence_before();
                }
                if (layer == 1) {
                    // h to global memory while the tensor cores run f's first layer
        #pragma unroll
                    for (int j = 0; j < decltype(nu)::value; ++j)
        #pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (hrow[j][i] >= 0) H[(size_t)hrow[j][i] * D + c] = hv[j][i];
                }
            }
            return true;
        };
        bool ok = true;
        PT_DECL(12);
        for (int level = 0; level < n_levels && ok; ++level) {
            const int slot = level % kRing;
            ok = wait_or_abort<true>(&bar_meta[slot], (level / kRing) & 1, abort);
            PT(0);
            if (level > 0) ok = ok && wait_or_abort<true>(&bar_level, (level - 1) & 1, abort);
            ok = __all_sync(0xffffffffu, ok);
            PT(1);
            if (!ok) break;
            rec = ring_rec(slot);
            nslot = ring_nslot(slot);
            xs = ring_x(slot);
            const int level_rows = ring_head(slot)[1];
            for (int r_base = 0; r_base < level_rows && ok; r_base += kTileRows) {
                const int R = min(kTileRows, level_rows - r_base);
                // most tiles have at most one 8-row unit per warp: the short code path
                ok = R <= 32 ? epilogue_tile(std::integral_constant<int, 1>(), r_base, R)
                             : epilogue_tile(std::integral_constant<int, 2>(), r_base, R);
            }
            PT(2);
            mbar_arrive(&bar_level);
            mbar_arrive(&bar_free[slot]);
        }
#ifdef PLACETO_PHASE_TIMERS
        if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0)
            printf("epilogue (cycles per level): wait staged level %lld, wait level barrier %lld, tiles %lld\n",
                   pt_[0] / n_levels, pt_[1] / n_levels, pt_[2] / n_levels);
#endif
    } else if (warp == kCtlWarp) {
        // ------------------------------------------------------------ control warp: one thread issues
        if (lane == 0) {
            const uint64_t a_desc = make_desc(smem_addr(sA), LBO_A, D * 32);
            const uint64_t b_desc = make_desc(smem_addr(sB), LBO_B, SBO_B);
            unsigned k_epi = 0;
            bool ok = true;
            PT_DECL(4);
            for (int level = 0; level < n_levels && ok; ++level) {
                const int slot = level % kRing;
                ok = wait_or_abort<true>(&bar_meta[slot], (level / kRing) & 1, abort);
                PT(0);
                if (!ok) break;
                const int level_rows = ring_head(slot)[1];
                for (int r_base = 0; r_base < level_rows && ok; r_base += kTileRows) {
                    const int R = min(kTileRows, level_rows - r_base);
                    const uint32_t idesc = make_idesc(128, 2 * ((R + 7) & ~7));
                    for (int layer = 0; layer < 4; ++layer) {
                        ok = wait_or_abort<true>(&bar_epi, k_epi++ & 1, abort);
                        if (!ok) break;
                        tc_fence_after();
                        PT(1);
                        // the address field of a descriptor counts 16-byte units
                        const uint64_t wa = a_desc + (uint64_t)(layer * (A_BYTES >> 4));
#pragma unroll
                        for (int ks = 0; ks < D / 8; ++ks)
                            mma_tf32(tmem, wa + (uint64_t)(ks * (2 * LBO_A >> 4)), b_desc + (uint64_t)(ks * (2 * LBO_B >> 4)),
                                     idesc, ks > 0);
                        mma_commit(&bar_mma);
                        PT(2);
                    }
                }
            }
            // whatever was issued has to finish before the tensor memory goes back
            mma_commit(&bar_drain);
            wait_or_abort<true>(&bar_drain, 0, abort);
#ifdef PLACETO_PHASE_TIMERS
            if (blockIdx.x == 0 && blockIdx.y == 0)
                printf("control (cycles per level): wait staged level %lld, wait operands %lld, issue %lld\n",
                       pt_[0] / n_levels, pt_[1] / n_levels, pt_[2] / n_levels);
#endif
        }
    } else {
        // ------------------------------------------------------------ loader warp
        const int4 *__restrict__ lvl4 = lv.lvl4;
        const int4 *__restrict__ pos4 = lv.pos4;
        const float *__restrict__ X = a.X;
        const int per_node = nb * F;
        const bool vec = (F & 3) == 0;
        const unsigned magic_nb = (unsigned)((0x100000000ull + nb - 1) / nb);
        bool ok = true;
        PT_DECL(2);
        for (int level = 0; level < n_levels && ok; ++level) {
            const int slot = level % kRing;
            if (level >= kRing) {
                ok = __all_sync(0xffffffffu, wait_or_abort<true>(&bar_free[slot], (level / kRing - 1) & 1, abort));
                if (!ok) break;
            }
            PT(0);
            const int4 L = lvl4[level];          // first position, width, first neighbour entry, entries
            int4 *rec = ring_rec(slot);
            int *nslot = ring_nslot(slot);
            float *xs = ring_x(slot);
            if (lane == 0) {
                ring_head(slot)[0] = L.y;
                ring_head(slot)[1] = L.y * nb;
            }
            for (int r = lane; r < L.y * nb; r += 32) {
                const int qp = nb == 1 ? r : (int)__umulhi((unsigned)r, magic_nb), s = r - qp * nb;
                const int4 m = pos4[L.x + qp];   // neighbour range, own slot, node id
                PLACETO_DEBUG_CHECK(a.status, m.x >= L.z && m.x <= m.y && m.y <= L.z + L.w && m.z >= -1 &&
                                                  m.z < lv.n_slots && m.w >= 0 && m.w < a.n && b_first + s < B);
                rec[r] = make_int4((m.x - L.z) | ((m.y - m.x) << 16), s, m.z >= 0 ? (m.z * S + s) * D : -1,
                                   m.w * B + b_first + s);
            }
            for (int e = lane; e < L.w; e += 32) {
                nslot[e] = lv.nbr_slot[L.z + e];
                PLACETO_DEBUG_CHECK(a.status, nslot[e] >= 0 && nslot[e] < lv.n_slots);
            }
            PLACETO_DEBUG_CHECK(a.status, L.x >= 0 && L.y >= 1 && L.x + L.y <= a.n && L.y <= a.max_level_width &&
                                              L.w <= lv.max_level_nbr);
            if (vec) {
                const int per4 = per_node >> 2;
                for (int i = lane; i < L.y * per4; i += 32) {
                    const int qp = i / per4, piece = i - qp * per4;
                    const int node = pos4[L.x + qp].w;
                    reinterpret_cast<float4 *>(xs)[i] =
                        reinterpret_cast<const float4 *>(X + ((size_t)node * B + b_first) * F)[piece];
                }
            } else {
                for (int i = lane; i < L.y * per_node; i += 32) {
                    const int qp = i / per_node, piece = i - qp * per_node;
                    const int node = pos4[L.x + qp].w;
                    xs[i] = X[((size_t)node * B + b_first) * F + piece];
                }
            }
            mbar_arrive(&bar_meta[slot]);
            PT(1);
        }
#ifdef PLACETO_PHASE_TIMERS
        if (blockIdx.x == 0 && blockIdx.y == 0 && lane == 0)
            printf("loader (cycles per level): wait free slot %lld, stage %lld\n", pt_[0] / n_levels, pt_[1] / n_levels);
#endif
    }
    if (abort_s && tid == 0) report_status(a.status, PLACETO_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == kCtlWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
}

bool relu2_64(const DevMlp &m, int in) {
    return m.n_layers == 2 && m.in_dim == in && m.hidden_dim == D && m.out_dim == D && m.act == 0 &&
           m.final_act == 1;
}

}  // namespace

bool embed_tc_applicable(const EmbedArgs &a) {
    if (a.d != D || a.F < 1 || a.F > 16) return false;
    for (int dir = 0; dir < 2; ++dir) {
        if (!relu2_64(a.f[dir], D + a.F) || !relu2_64(a.g[dir], D)) return false;
        if (a.lv[dir].lvl4 == nullptr || a.lv[dir].pos4 == nullptr) return false;
        if (a.lv[dir].max_level_nbr >= 32768) return false;      // a row record packs first entry and count into 16 bits each
    }
    return true;
}

cudaError_t launch_embed_tc(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap) {
    TcPlan p{};
    const int blocks_wanted = std::max(1, di.sm_count / 2);          // per direction
    const int want = std::max(1, std::min(a.B, blocks_wanted));
    p.S = (a.B + want - 1) / want;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 2048;   // static shared memory, alignment
    auto layout = [&](int S) {
        size_t off = 4 * (size_t)A_BYTES + B_BYTES;
        p.off_msg = (int)off;
        const int slots = std::max(a.lv[0].n_slots, a.lv[1].n_slots);
        off += (size_t)slots * S * D * sizeof(float);
        off = (off + 15) & ~(size_t)15;
        p.off_ring = (int)off;
        const int width = a.max_level_width;
        const int nbrs = std::max(a.lv[0].max_level_nbr, a.lv[1].max_level_nbr);
        size_t r = 16;                                   // the level's width and row count
        p.off_rec = (int)r;
        r += (size_t)width * S * sizeof(int4);
        p.off_nslot = (int)r;
        r += ((size_t)nbrs * sizeof(int) + 15) & ~(size_t)15;
        p.off_x = (int)r;
        r += ((size_t)width * S * a.F * sizeof(float) + 15) & ~(size_t)15;
        p.ring_bytes = (int)r;
        off += kRing * r;
        return off;
    };
    while (p.S > 1 && layout(p.S) > budget) --p.S;
    const size_t need = layout(p.S);
    if (need > budget) return cudaErrorNotSupported;
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.smem_bytes = (int)need;
    auto kern = embed_tc_kernel;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, p.smem_bytes);
    if (err != cudaSuccess) return err;
    err = launch_overlapped(overlap, kern, dim3(p.n_slices, 2), dim3(kThreads), (size_t)p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace placeto
