// One synchronous round of step 2 (Sec. 2.2 step 2 of the Placeto paper: all
// nodes updated at once from the previous round's values) specialised for
// d = 32 with two-layer ReLU networks of hidden width 32:
//   h_v = g( sum_{u in nbr(v)} m_u ),   m_v' = f([h_v || x_v]),
// m read from the previous round's buffer, m' written to the next one.
//
// Unlike the progressive sweep, every (node, state) row of a round is
// independent, so the kernel is a plain throughput loop: one persistent block
// per SM and direction half, lane j of every warp keeps column j of the
// direction's four weight matrices in registers, a warp takes two states of a
// node per pass (grid-stride over all such pairs), gathers the neighbours'
// messages from global memory (coalesced 128-byte rows, L2 resident), and runs
// the four layers exchanging the 32 outputs through a per-warp shared buffer
// read back as broadcast 128-bit loads. The shared loads bound it, as they bound
// the wide levels of the sweep kernel. With eight warps per SM nothing would hide
// the L2 latency of the gather, so the schedule (order, CSR) is staged in shared
// memory when it fits and the rows of the next pass (features, up to four
// neighbour messages per state) are loaded into registers before the current
// pass computes.
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kD = 32;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kAhead = 4;          // neighbour rows per state loaded one pass ahead

template <int K>
__device__ __forceinline__ void layer2(const float (&w)[K], float bias, const float *in, int stride,
                                       float (&out)[2]) {
    float acc[2][2] = {{bias, 0.f}, {bias, 0.f}};
#pragma unroll
    for (int k = 0; k < K; k += 4) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const float4 u = *reinterpret_cast<const float4 *>(in + r * stride + k);
            acc[r][0] = fmaf(u.x, w[k], acc[r][0]);
            acc[r][1] = fmaf(u.y, w[k + 1], acc[r][1]);
            acc[r][0] = fmaf(u.z, w[k + 2], acc[r][0]);
            acc[r][1] = fmaf(u.w, w[k + 3], acc[r][1]);
        }
    }
    out[0] = acc[0][0] + acc[0][1];
    out[1] = acc[1][0] + acc[1][1];
}

template <int F4>   // feature width padded to 4 * F4
__global__ void __launch_bounds__(kThreads, 1)
embed_rounds_d32_kernel(const EmbedArgs a, const float *__restrict__ Min0,
                        const float *__restrict__ Min1, float *__restrict__ Mout0,
                        float *__restrict__ Mout1, int first, int staged) {
    constexpr int KF = kD + 4 * F4;
    __shared__ __align__(16) float exch[kWarps][4 * KF];
    const int dir = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F, n = a.n;
    const DevMlp f = a.f[dir], g = a.g[dir];
    float g1[kD], g2[kD], f2[kD], f1[KF];
#pragma unroll
    for (int k = 0; k < kD; ++k) {
        g1[k] = g.W1[k * kD + lane];
        g2[k] = g.W2[k * kD + lane];
        f2[k] = f.W2[k * kD + lane];
    }
#pragma unroll
    for (int k = 0; k < KF; ++k) f1[k] = (k < kD + F) ? f.W1[k * kD + lane] : 0.f;
    const float bg1 = g.b1[lane], bg2 = g.b2[lane], bf1 = f.b1[lane], bf2 = f.b2[lane];
    const float *__restrict__ X = a.X;
    const float *__restrict__ Min = dir == 0 ? Min0 : Min1;
    float *__restrict__ Mout = dir == 0 ? Mout0 : Mout1;
    float *__restrict__ H = a.H[dir];
    float *A = exch[warp], *Bf = exch[warp] + 2 * KF;
    if (lane < KF - kD) {       // the padding behind the features stays zero
        A[kD + lane] = 0.f;
        A[KF + kD + lane] = 0.f;
    }
    // schedule in shared memory when the launcher found room for it
    extern __shared__ int sched[];
    const int *order = lv.order, *nbr_ptr = lv.nbr_ptr, *nbr = lv.nbr;
    if (staged) {
        for (int i = threadIdx.x; i < n; i += kThreads) sched[i] = lv.order[i];
        for (int i = threadIdx.x; i <= n; i += kThreads) sched[n + i] = lv.nbr_ptr[i];
        for (int i = threadIdx.x; i < lv.n_nbr; i += kThreads) sched[2 * n + 1 + i] = lv.nbr[i];
        order = sched; nbr_ptr = sched + n; nbr = sched + 2 * n + 1;
        __syncthreads();
    }
    const int ppn = (B + 1) >> 1;                       // state pairs per node
    const int items = n * ppn;                          // n * B < 2^31 is checked by the caller
    const int step = gridDim.x * kWarps;
    struct Pass {
        int pos, v, e0, e1, b0, b1;
        bool two;
        float x0, x1, t[kAhead][2];
    };
    // issues the loads of one pass: features and the first kAhead neighbour rows
    auto fetch = [&](int item, Pass &p) {
        p.pos = (int)((unsigned)item / (unsigned)ppn);
        p.b0 = (item - p.pos * ppn) * 2;
        p.two = p.b0 + 1 < B;
        p.b1 = p.two ? p.b0 + 1 : p.b0;
        p.v = order[p.pos];
        p.e0 = nbr_ptr[p.pos];
        p.e1 = nbr_ptr[p.pos + 1];
        p.x0 = lane < F ? X[((size_t)p.v * B + p.b0) * F + lane] : 0.f;
        p.x1 = lane < F ? X[((size_t)p.v * B + p.b1) * F + lane] : 0.f;
#pragma unroll
        for (int k = 0; k < kAhead; ++k) {
            p.t[k][0] = 0.f;
            p.t[k][1] = 0.f;
            if (!first && p.e0 + k < p.e1) {
                const size_t row = (size_t)nbr[p.e0 + k] * B;
                p.t[k][0] = Min[(row + p.b0) * kD + lane];
                p.t[k][1] = Min[(row + p.b1) * kD + lane];
            }
        }
    };
    int item = blockIdx.x * kWarps + warp;
    Pass cur, nxt;
    if (item < items) fetch(item, cur);
    for (; item < items; item += step) {
        if (item + step < items) fetch(item + step, nxt);
        const int v = cur.v, b0 = cur.b0, b1 = cur.b1;
        const bool two = cur.two;
        float acc[2] = {0.f, 0.f};
        if (!first) {
#pragma unroll
            for (int k = 0; k < kAhead; ++k) {
                acc[0] += cur.t[k][0];
                acc[1] += cur.t[k][1];
            }
            for (int e = cur.e0 + kAhead; e < cur.e1; ++e) {    // further neighbours, ascending
                const size_t row = (size_t)nbr[e] * B;
                acc[0] += Min[(row + b0) * kD + lane];
                acc[1] += Min[(row + b1) * kD + lane];
            }
            __syncwarp();                   // the previous pass has read A and Bf
            A[lane] = acc[0];
            A[KF + lane] = acc[1];
            __syncwarp();
            layer2<kD>(g1, bg1, A, KF, acc);
            Bf[lane] = fmaxf(acc[0], 0.f);
            Bf[KF + lane] = fmaxf(acc[1], 0.f);
            __syncwarp();
            layer2<kD>(g2, bg2, Bf, KF, acc);
            acc[0] = fmaxf(acc[0], 0.f);
            acc[1] = fmaxf(acc[1], 0.f);
            H[((size_t)v * B + b0) * kD + lane] = acc[0];
            if (two) H[((size_t)v * B + b1) * kD + lane] = acc[1];
        }
        __syncwarp();
        A[lane] = acc[0];                   // [h || x]; h = 0 before the first round
        A[KF + lane] = acc[1];
        if (lane < F) {
            A[kD + lane] = cur.x0;
            A[KF + kD + lane] = cur.x1;
        }
        __syncwarp();
        layer2<KF>(f1, bf1, A, KF, acc);
        Bf[lane] = fmaxf(acc[0], 0.f);
        Bf[KF + lane] = fmaxf(acc[1], 0.f);
        __syncwarp();
        layer2<kD>(f2, bf2, Bf, KF, acc);
        Mout[((size_t)v * B + b0) * kD + lane] = fmaxf(acc[0], 0.f);
        if (two) Mout[((size_t)v * B + b1) * kD + lane] = fmaxf(acc[1], 0.f);
        cur = nxt;
    }
}

}  // namespace

cudaError_t launch_embed_rounds_d32(const EmbedArgs &a, const DeviceInfo &di, int rounds,
                                    float *const msg[4], cudaStream_t stream) {
    void (*kern)(const EmbedArgs, const float *, const float *, float *, float *, int, int) = nullptr;
    switch ((a.F + 3) / 4) {
        case 1: kern = embed_rounds_d32_kernel<1>; break;
        case 2: kern = embed_rounds_d32_kernel<2>; break;
        case 3: kern = embed_rounds_d32_kernel<3>; break;
        case 4: kern = embed_rounds_d32_kernel<4>; break;
        default: return cudaErrorNotSupported;
    }
    const long long items = (long long)a.n * ((a.B + 1) / 2);
    const int per_dir = std::max(1, di.sm_count / 2);
    const int blocks = (int)std::max(1LL, std::min<long long>(per_dir, (items + kWarps - 1) / kWarps));
    // the schedule of the larger direction in shared memory, if it fits beside the exchange buffers
    const size_t sched_bytes = (2 * (size_t)a.n + 1 + std::max(a.lv[0].n_nbr, a.lv[1].n_nbr)) * sizeof(int);
    const int staged = sched_bytes <= 160 * 1024 ? 1 : 0;
    const size_t smem = staged ? sched_bytes : 0;
    cudaError_t attr = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (attr != cudaSuccess) return attr;
    for (int r = 0; r <= rounds; ++r) {
        const float *in0 = msg[(r + 1) & 1], *in1 = msg[2 + ((r + 1) & 1)];
        float *out0 = msg[r & 1], *out1 = msg[2 + (r & 1)];
        kern<<<dim3(blocks, 2), kThreads, smem, stream>>>(a, in0, in1, out0, out1, r == 0 ? 1 : 0, staged);
        count_launch();
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

}  // namespace placeto
