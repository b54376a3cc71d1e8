// Step 3 of the policy (Sec. 2.2 step 3 of the Placeto paper) for d = 64 on the
// fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
// partial sums over a chunk of nodes of
//   l_i(e_u) = relu(W_i^T e_u + b_i),  e_u = [h_down_u || h_up_u || x_u],  i = set of u relative to cur[b],
// in the layout the head kernel adds up. The rows (node, state) have no
// dependency on one another, so unlike the sweep this is a throughput problem:
// about 1.1 M rows of 140 -> 64 on the NASNet-shaped workload.
//
// Arithmetic: as in the tcgen05 sweep kernel the product is computed transposed
// with TF32 operands split into head and tail. The instruction's M = 128 rows
// are W_i^T's head and tail rows (rows 32q + j / 32q + 16 + j: head / tail of
// output column 16q + j), its N = 128 columns a tile's 64 data rows twice
// (heads, then tails), so one instruction per 8-wide k-step yields all four
// partial products. The stacked weights of the current set live in tensor
// memory (the A operand is read from there), which leaves shared memory to two
// operand tiles.
//
// Work: an item is (state b, chunk of nodes); the block walks its items once per
// set (three passes, so the weights in tensor memory change twice), and per
// item and set the chunk's nodes of that set, in ascending order, 64 per tile.
// Roles, connected by mbarriers with bounded waits:
//   - sixteen producer warps gather the tile's rows from H_down, H_up and X (a warp
//     per row: 256 + 256 + 4F contiguous bytes), split them and store them in
//     the operand layout; a four-deep ring of tile descriptors (rows, flags,
//     item) travels with the tiles; the node list of a (set, item) pair is compacted by all
//     producer warps a pair ahead;
//   - one thread issues the instructions of a tile into one of two accumulators
//     and commits them to the barriers that free the tile and hand the
//     accumulator over;
//   - four epilogue warps (one per quadrant of tensor memory) add the four
//     partial products, apply bias and ReLU and keep the running sum of the
//     item; at the item's last tile the sum goes to the partial-sum array.
// Summation order is fixed (ascending node id per thread, then a fixed
// combination), so results are reproducible bit for bit.
#include <algorithm>
#include <cstdio>

#include "kernels.cuh"

namespace placeto {

namespace {

// Build with -DPLACETO_PHASE_TIMERS to have block 0 print, per role, the cycles it spent in
// each phase (sums over the launch, from clock64()).
#ifdef PLACETO_PHASE_TIMERS
#define PT_DECL(n) long long pt_[n] = {}; long long pt_last_ = clock64()
#define PT(i) do { const long long pt_now_ = clock64(); pt_[i] += pt_now_ - pt_last_; pt_last_ = pt_now_; } while (0)
#else
#define PT_DECL(n) do { } while (0)
#define PT(i) do { } while (0)
#endif

constexpr int kD = 64;
constexpr int kTileRows = 64;
constexpr int kEpiWarps = 4, kProdWarps = 16;
constexpr int kIssueWarp = kEpiWarps + kProdWarps;
constexpr int kThreads = (kIssueWarp + 1) * 32;
constexpr int kProdThreads = kProdWarps * 32, kEpiThreads = kEpiWarps * 32;
constexpr int kStages = 2, kMetaRing = 4;
constexpr int kMaxScan = 4;                            // 32-node steps of a warp's slice of a chunk
constexpr int kRowsPerWarp = kTileRows / kProdWarps;   // a producer warp's rows of a tile
constexpr int LBO = 144;                      // bytes between the 16-byte k-chunks of 8 rows (16 B of padding)
constexpr int kGroups = 2 * kTileRows / 8;    // groups of 8 operand rows per tile
constexpr int kTmemCols = 512;
constexpr int kAccCol = 160;                  // accumulators at columns 160 and 288, the weights below
constexpr int kLastOfItem = 1, kLastOfSet = 2;

struct PoolTcPlan {
    int chunk_nodes, chunks, items;
    int K;                 // inner width: 2 d + F rounded up to 8
    int tile_bytes;        // one operand tile
    int off_list;          // byte offset of the node lists
    int off_rel;           // byte offset of the cached relation rows, or -1: scanned in global memory
    int smem_bytes;
};

__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
__device__ __forceinline__ uint32_t make_idesc(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem] * B[shared memory descriptor]
__device__ __forceinline__ void mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accum) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Bounded wait; gives up early when another thread has raised *abort. Each try may park the
// thread for the hardware's default time limit, so a waiting warp takes few issue slots.
__device__ __forceinline__ bool wait_or_abort(unsigned long long *bar, unsigned parity, volatile int *abort) {
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
    *abort = 1;
    return false;
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ unsigned tf32_round(float x) { return (__float_as_uint(x) + 0x1000u) & 0xffffe000u; }

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
__device__ __forceinline__ void tmem_st8(uint32_t ta, const uint32_t (&a)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(a[0]), "r"(a[1]),
                 "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]), "r"(ta)
                 : "memory");
}

// Four values of a row -> head and tail chunks of the operand tile. The head is rounded to
// TF32 here; the tail x - head is exact in FP32 and goes in as it is: the tensor core reads
// its upper 19 bits, and what that drops is below 2^-22 of x.
__device__ __forceinline__ void store_split4(unsigned char *head_at, int tail_bytes, float4 v) {
    float4 h, t;
    h.x = __uint_as_float(tf32_round(v.x)); t.x = v.x - h.x;
    h.y = __uint_as_float(tf32_round(v.y)); t.y = v.y - h.y;
    h.z = __uint_as_float(tf32_round(v.z)); t.z = v.z - h.z;
    h.w = __uint_as_float(tf32_round(v.w)); t.w = v.w - h.w;
    *reinterpret_cast<float4 *>(head_at) = h;
    *reinterpret_cast<float4 *>(head_at + tail_bytes) = t;
}

__global__ void __launch_bounds__(kThreads, 1) pool_tc_kernel(const PoolArgs a, const PoolTcPlan p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ unsigned long long bar_full[kStages], bar_buf_free[kStages], bar_acc_full[kStages], bar_acc_free[kStages];
    __shared__ unsigned long long bar_a_ready, bar_drain;
    __shared__ int4 meta[kMetaRing];            // {rows, flags, state, chunk}
    __shared__ int warp_count[2][kProdWarps];
    __shared__ uint32_t tmem_s;
    __shared__ int abort_s;
    dependents_may_start();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = a.n, B = a.B, F = a.F;
    const int E = 2 * kD + F, K = p.K, KC = K / 4, SBO = KC * LBO;
    const int tail_bytes = (kGroups / 2) * SBO;          // tails sit 64 operand rows behind the heads
    unsigned char *tiles = smem;
    int *list = reinterpret_cast<int *>(smem + p.off_list);

    if (warp == kIssueWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_s)),
                     "n"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bar_full[s], kProdThreads);
            mbar_init(&bar_buf_free[s], 1);
            mbar_init(&bar_acc_full[s], 1);
            mbar_init(&bar_acc_free[s], kEpiThreads);
        }
        mbar_init(&bar_a_ready, kEpiThreads);
        mbar_init(&bar_drain, 1);
        abort_s = 0;
    }
    // operand tiles start at zero: the padding chunks behind the 2 d + F real columns stay zero for good
    for (int i = tid; i < kStages * p.tile_bytes / 16; i += kThreads)
        reinterpret_cast<float4 *>(tiles)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_s;
    volatile int *abort = &abort_s;
    const int first_item = blockIdx.x, item_step = gridDim.x;
    // The walk over (set, item) pairs, flattened: pair k = set * my_items + j.
    const int my_items = (p.items - first_item + item_step - 1) / item_step;
    const int n_pairs = 3 * my_items;

    if (warp < kEpiWarps) {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp;
        const bool lo = lane < 16;
        const int c = 16 * q + (lane & 15), r_add = lo ? 0 : 4;
        const uint32_t lane_base = tmem + ((uint32_t)(32 * q) << 16);
        unsigned tc = 0;
        bool ok = true;
        PT_DECL(4);
        for (int set = 0; set < 3 && ok; ++set) {
            // this lane's row of the stacked weights: head (lanes 0..15) or tail of column c
            const float *W = a.l[set].W1;
            for (int k0 = 0; k0 < K; k0 += 8) {
                uint32_t v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float w = k0 + j < E ? W[(size_t)(k0 + j) * kD + c] : 0.f;
                    const unsigned h = tf32_round(w);
                    v[j] = lo ? h : tf32_round(w - __uint_as_float(h));
                }
                tmem_st8(lane_base + k0, v);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            mbar_arrive(&bar_a_ready);
            const float bias = a.l[set].b1[c];
            float sum = 0.f;
            PT(0);
            for (;;) {
                const int acc = tc & 1;
                ok = __all_sync(0xffffffffu, wait_or_abort(&bar_acc_full[acc], (tc >> 1) & 1, abort));
                if (!ok) break;
                tc_fence_after();
                PT(1);
                const int4 m = meta[tc % kMetaRing];
                const uint32_t d_col = lane_base + kAccCol + acc * 128;
                for (int u = 0; 8 * u < m.x; ++u) {
                    uint32_t ha[8], ta[8];
                    tmem_ld8x2(d_col + 8 * u, d_col + kTileRows + 8 * u, ha, ta);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        // lanes below 16 hold head-weight products, the others tail-weight products;
                        // each half finishes four of the unit's eight rows
                        const float first = __uint_as_float(ha[i]) + __uint_as_float(ta[i]);
                        const float second = __uint_as_float(ha[4 + i]) + __uint_as_float(ta[4 + i]);
                        const float v = (lo ? first : second) + __shfl_xor_sync(0xffffffffu, lo ? second : first, 16);
                        if (8 * u + i + r_add < m.x) sum += fmaxf(v + bias, 0.f);
                    }
                }
                tc_fence_before();
                mbar_arrive(&bar_acc_free[acc]);
                ++tc;
                if (m.y & kLastOfItem) {
                    const float total = sum + __shfl_xor_sync(0xffffffffu, sum, 16);
                    if (lo) a.partial[(((size_t)m.w * B + m.z) * 3 + set) * kD + c] = total;
                    sum = 0.f;
                }
                PT(2);
                if (m.y & kLastOfSet) break;
            }
        }
#ifdef PLACETO_PHASE_TIMERS
        if (blockIdx.x == 0 && tid == 0)
            printf("epilogue (cycles per tile, %u tiles): weights to tensor memory %lld (total), wait accumulator %lld, sums %lld\n",
                   tc, pt_[0], pt_[1] / tc, pt_[2] / tc);
#endif
    } else if (warp < kIssueWarp) {
        // ------------------------------------------------------------ producer warps
        const int pw = warp - kEpiWarps, ptid = tid - kEpiThreads;
        const int f4 = F >> 2;
        dependency_wait();          // the embeddings may come from a kernel that is still running
        // An item's row of the relation matrix is scanned once per set: keep the block's rows in
        // shared memory when they fit.
        uint8_t *rel_cache = p.off_rel >= 0 ? smem + p.off_rel : nullptr;
        if (rel_cache != nullptr) {
            for (int j = 0; j < my_items; ++j) {
                const int item = first_item + j * item_step;
                const int b = item % B, chunk = item / B;
                const int u0 = chunk * p.chunk_nodes, nu = min(n, u0 + p.chunk_nodes) - u0;
                const int cur = a.cur[b];
                const bool valid = cur >= 0 && cur < n;
                for (int u = ptid; u < nu; u += kProdThreads)
                    rel_cache[j * p.chunk_nodes + u] = valid ? a.relation[(size_t)cur * n + u0 + u] : 3;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kProdThreads) : "memory");
        }
        // Node list of pair k (the chunk's nodes of the set, ascending), built by all producer
        // warps a pair ahead into the other of two buffers: every warp compacts its slice.
        auto build_list = [&](int k, int *out, int *count) {
            const int set = k / my_items, item = first_item + (k % my_items) * item_step;
            const int b = item % B, chunk = item / B;
            const int u0 = chunk * p.chunk_nodes, nu = min(n, u0 + p.chunk_nodes) - u0;
            const int cur = a.cur[b];
            const bool valid = cur >= 0 && cur < n;
            PLACETO_DEBUG_CHECK(a.status, valid);
            const uint8_t *rel = rel_cache != nullptr ? rel_cache + (k % my_items) * p.chunk_nodes
                                                      : a.relation + (size_t)(valid ? cur : 0) * n + u0;
            const int per_warp = (((nu + kProdWarps - 1) / kProdWarps) + 31) & ~31;
            const int w0 = min(nu, pw * per_warp), w1 = min(nu, w0 + per_warp);
            unsigned masks[kMaxScan];           // at most kMaxScan 32-node steps per warp (the chunk size is capped)
            int mine = 0;
#pragma unroll
            for (int i = 0; i < kMaxScan; ++i) {
                const int u = w0 + 32 * i + lane;
                masks[i] = __ballot_sync(0xffffffffu, valid && u < w1 && rel[u] == set);
                mine += __popc(masks[i]);
            }
            if (lane == 0) warp_count[k & 1][pw] = mine;
            asm volatile("bar.sync 1, %0;" ::"n"(kProdThreads) : "memory");
            int at = 0, cnt = 0;
            for (int w = 0; w < kProdWarps; ++w) {
                const int c = warp_count[k & 1][w];
                if (w < pw) at += c;
                cnt += c;
            }
#pragma unroll
            for (int i = 0; i < kMaxScan; ++i) {
                if (masks[i] >> lane & 1) out[at + __popc(masks[i] & ((1u << lane) - 1))] = u0 + w0 + 32 * i + lane;
                at += __popc(masks[i]);
            }
            *count = cnt;
        };
        int *lists[2] = {list, list + p.chunk_nodes};
        // a warp's rows of a tile: r = pw + j * kProdWarps. The embeddings take a warp per row
        // (lanes 0..15 the 16-byte pieces of h_down, 16..31 of h_up); the raw features of all
        // the warp's rows go in one pass, lane = (row j, piece) for lane < kRowsPerWarp * F / 4.
        // The rows of the next tile are requested right after a tile has been stored and
        // fenced (the fence would wait for loads in flight) and arrive while the warp waits
        // for a free tile.
        float4 hv[kRowsPerWarp], xv;
        const int xj = lane / f4, xpiece = lane - xj * f4;      // f4 <= 4: lanes 0 .. 4 f4 - 1 are in use
        auto prefetch = [&](const int *rows_of_tile, int rows, int b) {
#pragma unroll
            for (int j = 0; j < kRowsPerWarp; ++j) {
                const int r = pw + j * kProdWarps;
                if (r < rows) {
                    const size_t row = (size_t)rows_of_tile[r] * B + b;
                    hv[j] = reinterpret_cast<const float4 *>(a.H[lane >> 4] + row * kD)[lane & 15];
                }
            }
            const int rx = pw + xj * kProdWarps;
            if (xj < kRowsPerWarp && rx < rows)
                xv = reinterpret_cast<const float4 *>(a.X + ((size_t)rows_of_tile[rx] * B + b) * F)[xpiece];
        };
        unsigned tc = 0;
        bool ok = true;
        PT_DECL(4);
        int cnt = 0, cnt_next = 0;
        build_list(0, lists[0], &cnt);
        asm volatile("bar.sync 1, %0;" ::"n"(kProdThreads) : "memory");       // list 0 complete
        prefetch(lists[0], min(kTileRows, cnt), first_item % B);
        // After a time-out (ok == false) the warp keeps walking the same loops without touching
        // tiles or barriers of the pipeline: every producer warp has to reach the named barriers.
        for (int k = 0; k < n_pairs; ++k) {
            const int item = first_item + (k % my_items) * item_step;
            const int b = item % B, chunk = item / B;
            const int *cur_list = lists[k & 1];
            // the next pair's list, while the first tile's rows are on their way
            if (k + 1 < n_pairs) build_list(k + 1, lists[(k + 1) & 1], &cnt_next);
            asm volatile("bar.sync 1, %0;" ::"n"(kProdThreads) : "memory");   // next list complete
            PT(0);
            const int n_tiles = max(1, (cnt + kTileRows - 1) / kTileRows);
            for (int t = 0; t < n_tiles; ++t) {
                const int stage = tc & 1;
                if (ok && tc >= kStages)
                    ok = __all_sync(0xffffffffu, wait_or_abort(&bar_buf_free[stage], ((tc >> 1) - 1) & 1, abort));
                PT(1);
                const int rows = max(0, min(kTileRows, cnt - t * kTileRows));
                if (ok) {
                    unsigned char *tile = tiles + stage * p.tile_bytes;
#pragma unroll
                    for (int j = 0; j < kRowsPerWarp; ++j) {
                        const int r = pw + j * kProdWarps;
                        if (r < rows) store_split4(tile + (r >> 3) * SBO + (r & 7) * 16 + lane * LBO, tail_bytes, hv[j]);
                    }
                    const int rx = pw + xj * kProdWarps;
                    if (xj < kRowsPerWarp && rx < rows)
                        store_split4(tile + (rx >> 3) * SBO + (rx & 7) * 16 + (32 + xpiece) * LBO, tail_bytes, xv);
                    if (ptid == 0) {
                        int flags = 0;
                        if (t == n_tiles - 1) flags |= kLastOfItem | ((k + 1) % my_items == 0 ? kLastOfSet : 0);
                        meta[tc % kMetaRing] = make_int4(rows, flags, b, chunk);
                    }
                    fence_async_smem();
                    mbar_arrive(&bar_full[stage]);
                }
                ++tc;
                // the rows of the tile after this one: of this pair, or the first of the next pair
                if (t + 1 < n_tiles) {
                    prefetch(cur_list + (t + 1) * kTileRows, min(kTileRows, cnt - (t + 1) * kTileRows), b);
                } else if (k + 1 < n_pairs) {
                    const int next_item = first_item + ((k + 1) % my_items) * item_step;
                    prefetch(lists[(k + 1) & 1], min(kTileRows, cnt_next), next_item % B);
                }
                PT(2);
            }
            cnt = cnt_next;
        }
#ifdef PLACETO_PHASE_TIMERS
        if (blockIdx.x == 0 && ptid == 0)
            printf("producer (cycles per tile, %u tiles): node lists %lld, wait free tile %lld, split + store + next loads %lld\n",
                   tc, pt_[0] / tc, pt_[1] / tc, pt_[2] / tc);
#endif
    } else if (warp == kIssueWarp && lane == 0) {
        // ------------------------------------------------------------ the issuing thread
        const uint32_t idesc = make_idesc(128, 2 * kTileRows);
        const int KS = K / 8;
        unsigned tc = 0;
        bool ok = true;
        PT_DECL(4);
        for (int set = 0; set < 3 && ok; ++set) {
            ok = wait_or_abort(&bar_a_ready, set & 1, abort);
            if (!ok) break;
            tc_fence_after();
            for (;;) {
                const int stage = tc & 1;
                PT(0);
                ok = wait_or_abort(&bar_full[stage], (tc >> 1) & 1, abort);
                PT(1);
                if (ok && tc >= kStages) ok = wait_or_abort(&bar_acc_free[stage], ((tc >> 1) - 1) & 1, abort);
                if (!ok) break;
                tc_fence_after();
                PT(2);
                const int4 m = meta[tc % kMetaRing];
                if (m.x > 0) {
                    const uint64_t b_desc = make_desc(smem_addr(tiles + stage * p.tile_bytes), LBO, SBO);
                    const uint32_t d_tmem = tmem + kAccCol + stage * 128;
                    for (int ks = 0; ks < KS; ++ks)
                        mma_tf32_ts(d_tmem, tmem + 8 * ks, b_desc + (uint64_t)(ks * (2 * LBO >> 4)), idesc, ks > 0);
                }
                mma_commit(&bar_buf_free[stage]);
                mma_commit(&bar_acc_full[stage]);
                ++tc;
                PT(3);
                if (m.y & kLastOfSet) break;
            }
        }
#ifdef PLACETO_PHASE_TIMERS
        if (blockIdx.x == 0)
            printf("issuer (cycles per tile, %u tiles): wait tile %lld, wait accumulator %lld, issue + commit %lld, other %lld\n",
                   tc, pt_[1] / tc, pt_[2] / tc, pt_[3] / tc, pt_[0] / tc);
#endif
        // whatever was issued has to finish before the tensor memory goes back
        mma_commit(&bar_drain);
        wait_or_abort(&bar_drain, 0, abort);
    }
    if (abort_s && tid == 0) report_status(a.status, PLACETO_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == kIssueWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
}

bool relu1x64(const DevMlp &m, int in) {
    return m.n_layers == 1 && m.in_dim == in && m.out_dim == kD && m.act == 0 && m.final_act == 1;
}

}  // namespace

bool pool_tc_applicable(const PoolArgs &a) {
    if (a.d != kD || a.F < 4 || a.F > 16 || (a.F & 3)) return false;
    for (int i = 0; i < 3; ++i)
        if (!relu1x64(a.l[i], 2 * kD + a.F)) return false;
    return true;
}

// Items are (state, chunk of nodes): enough of them to balance the persistent blocks, chunks
// of at least two tiles.
void pool_tc_chunks(int n, int B, const DeviceInfo &di, int *chunk_nodes, int *chunks) {
    int c = (6 * di.sm_count + B - 1) / B;
    c = std::max(1, std::min(c, n / (2 * kTileRows)));
    const int cap = kMaxScan * 32 * kProdWarps;            // a producer warp scans at most kMaxScan x 32 nodes
    c = std::max(c, (n + cap - 1) / cap);
    *chunk_nodes = (n + c - 1) / c;
    *chunks = (n + *chunk_nodes - 1) / *chunk_nodes;
}

cudaError_t launch_pool_tc(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap) {
    PoolTcPlan p{};
    p.chunk_nodes = a.chunk_nodes;
    p.chunks = a.chunks;
    p.items = a.B * a.chunks;
    p.K = (2 * kD + a.F + 7) & ~7;
    p.tile_bytes = kGroups * (p.K / 4) * LBO;
    p.off_list = kStages * p.tile_bytes;
    p.smem_bytes = p.off_list + ((2 * p.chunk_nodes * (int)sizeof(int) + 15) & ~15);
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 2048;
    if ((size_t)p.smem_bytes > budget) return cudaErrorNotSupported;
    const int grid = std::max(1, std::min(di.sm_count, p.items));
    const size_t rel_bytes = ((size_t)((p.items + grid - 1) / grid) * p.chunk_nodes + 15) & ~(size_t)15;
    p.off_rel = -1;
    if (p.smem_bytes + rel_bytes <= budget) {
        p.off_rel = p.smem_bytes;
        p.smem_bytes += (int)rel_bytes;
    }
    cudaError_t err = cudaFuncSetAttribute(pool_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, p.smem_bytes);
    if (err != cudaSuccess) return err;
    err = launch_overlapped(overlap, pool_tc_kernel, dim3(grid), dim3(kThreads), (size_t)p.smem_bytes, stream, a, p);
    count_launch();
    return err;
}

}  // namespace placeto
