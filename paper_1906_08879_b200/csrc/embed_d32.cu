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
//     buffer and read back as broadcast 128-bit loads: 4 FMAs per shared load.
//   - Two rows are in flight per warp for instruction-level parallelism.
//   - Messages never leave the SM: m_u lives in a shared-memory slot from the
//     level of u until its last consumer's level (slots assigned on the host).
//     Global traffic is the compulsory part only: read x, write h.
//   - The level schedule (order, CSR, slots) is staged in shared memory.
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
    int ints_in_smem;
    size_t smem_bytes;
};

// o0/o1 = bias + in0/in1 . w  over K inputs read as broadcast float4 from shared memory.
template <int K>
__device__ __forceinline__ void matvec2(const float (&w)[K], float bias, const float *in0,
                                        const float *in1, float &o0, float &o1) {
    float a0 = bias, a1 = 0.f, b0 = bias, b1 = 0.f;
#pragma unroll
    for (int k = 0; k < K; k += 4) {
        const float4 u = *reinterpret_cast<const float4 *>(in0 + k);
        const float4 v = *reinterpret_cast<const float4 *>(in1 + k);
        a0 = fmaf(u.x, w[k], a0);
        b0 = fmaf(v.x, w[k], b0);
        a1 = fmaf(u.y, w[k + 1], a1);
        b1 = fmaf(v.y, w[k + 1], b1);
        a0 = fmaf(u.z, w[k + 2], a0);
        b0 = fmaf(v.z, w[k + 2], b0);
        a1 = fmaf(u.w, w[k + 3], a1);
        b1 = fmaf(v.w, w[k + 3], b1);
    }
    o0 = a0 + a1;
    o1 = b0 + b1;
}

template <int F4>   // feature width padded to 4 * F4
__global__ void __launch_bounds__(kThreads, 1)
embed_d32_kernel(const EmbedArgs a, const D32Plan p) {
    constexpr int KF = kD + 4 * F4;      // padded input width of f's first layer
    extern __shared__ __align__(16) float smem[];
    const int dir = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const DevLevels lv = a.lv[dir];
    const int B = a.B, F = a.F;
    const int b_first = blockIdx.x * p.S;
    const int nb = min(p.S, B - b_first);

    // ---- shared memory: [schedule ints][message slots][per-warp exchange buffers]
    const int *level_ptr = lv.level_ptr, *order = lv.order, *nbr_ptr = lv.nbr_ptr;
    const int *nbr_slot = lv.nbr_slot, *own_slot = lv.own_slot;
    float *fsm = smem;
    if (p.ints_in_smem) {
        int *ism = reinterpret_cast<int *>(smem);
        auto stage = [&](const int *src, int count) {
            int *dst = ism;
            for (int i = threadIdx.x; i < count; i += kThreads) dst[i] = src[i];
            ism += (count + 3) & ~3;
            return (const int *)dst;
        };
        level_ptr = stage(lv.level_ptr, lv.n_levels + 1);
        order = stage(lv.order, a.n);
        nbr_ptr = stage(lv.nbr_ptr, a.n + 1);
        own_slot = stage(lv.own_slot, a.n);
        nbr_slot = stage(lv.nbr_slot, lv.n_nbr);
        fsm = reinterpret_cast<float *>(ism);
    }
    float *msg = fsm;                                       // [n_slots][S][32]
    float *xbuf = msg + (size_t)lv.n_slots * p.S * kD + (size_t)warp * 4 * KF;
    float *A0 = xbuf, *A1 = xbuf + KF, *B0 = xbuf + 2 * KF, *B1 = xbuf + 3 * KF;

    // ---- this lane's weight columns
    const DevMlp f = a.f[dir], g = a.g[dir];
    float wg1[kD], wg2[kD], wf1[KF], wf2[kD];
#pragma unroll
    for (int k = 0; k < kD; ++k) {
        wg1[k] = g.W1[k * kD + lane];
        wg2[k] = g.W2[k * kD + lane];
        wf2[k] = f.W2[k * kD + lane];
    }
#pragma unroll
    for (int k = 0; k < KF; ++k) wf1[k] = (k < kD + F) ? f.W1[k * kD + lane] : 0.f;
    const float bg1 = g.b1[lane], bg2 = g.b2[lane], bf1 = f.b1[lane], bf2 = f.b2[lane];
    const float *__restrict__ X = a.X;
    float *__restrict__ H = a.H[dir];
    __syncthreads();

    for (int level = 0; level < lv.n_levels; ++level) {
        const int p0 = level_ptr[level];
        const int rows = (level_ptr[level + 1] - p0) * nb;
        for (int r = 2 * warp; r < rows; r += 2 * kWarps) {
            // rows r and r + 1 (the second may not exist: it then repeats the first)
            const bool two = r + 1 < rows;
            const int q0 = r / nb, s0 = r - q0 * nb;
            const int r1 = two ? r + 1 : r;
            const int q1 = r1 / nb, s1 = r1 - q1 * nb;
            const int pos0 = p0 + q0, pos1 = p0 + q1;
            const int v0 = order[pos0], v1 = order[pos1];
            const size_t row0 = (size_t)v0 * B + b_first + s0, row1 = (size_t)v1 * B + b_first + s1;
            // raw features, needed at the third layer: issue the loads first
            float x0 = 0.f, x1 = 0.f;
            if (lane < F) { x0 = X[row0 * F + lane]; x1 = X[row1 * F + lane]; }
            // gather: sum of the neighbours' messages (column `lane`)
            float g0 = 0.f, g1 = 0.f;
            for (int e = nbr_ptr[pos0]; e < nbr_ptr[pos0 + 1]; ++e)
                g0 += msg[((size_t)nbr_slot[e] * p.S + s0) * kD + lane];
            for (int e = nbr_ptr[pos1]; e < nbr_ptr[pos1 + 1]; ++e)
                g1 += msg[((size_t)nbr_slot[e] * p.S + s1) * kD + lane];
            A0[lane] = g0; A1[lane] = g1;
            __syncwarp();
            float t0, t1;
            matvec2<kD>(wg1, bg1, A0, A1, t0, t1);
            B0[lane] = fmaxf(t0, 0.f); B1[lane] = fmaxf(t1, 0.f);
            __syncwarp();
            matvec2<kD>(wg2, bg2, B0, B1, t0, t1);
            t0 = fmaxf(t0, 0.f); t1 = fmaxf(t1, 0.f);
            H[row0 * kD + lane] = t0;
            if (two) H[row1 * kD + lane] = t1;
            const int slot0 = own_slot[pos0], slot1 = own_slot[pos1];
            if (slot0 >= 0 || slot1 >= 0) {          // somebody consumes the message
                A0[lane] = t0; A1[lane] = t1;
                if (lane < 4 * F4) { A0[kD + lane] = x0; A1[kD + lane] = x1; }
                __syncwarp();
                matvec2<KF>(wf1, bf1, A0, A1, t0, t1);
                B0[lane] = fmaxf(t0, 0.f); B1[lane] = fmaxf(t1, 0.f);
                __syncwarp();
                matvec2<kD>(wf2, bf2, B0, B1, t0, t1);
                if (slot0 >= 0) msg[((size_t)slot0 * p.S + s0) * kD + lane] = fmaxf(t0, 0.f);
                if (two && slot1 >= 0) msg[((size_t)slot1 * p.S + s1) * kD + lane] = fmaxf(t1, 0.f);
            }
        }
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

cudaError_t launch_embed_d32(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream) {
    D32Plan p;
    const int target = std::max(1, di.sm_count / 2);            // blocks per direction
    const int want = std::max(1, std::min(a.B, target));
    p.S = (a.B + want - 1) / want;
    const int F4 = (a.F + 3) / 4;
    const int KF = kD + 4 * F4;
    const size_t budget = (size_t)std::min(di.max_smem_optin, 227 * 1024) - 1024;
    const int max_slots = std::max(a.lv[0].n_slots, a.lv[1].n_slots);
    size_t ints = 0;
    for (int dir = 0; dir < 2; ++dir) {
        const DevLevels &lv = a.lv[dir];
        size_t s = ((lv.n_levels + 1 + 3) & ~3) + 2 * ((a.n + 3) & ~3) + ((a.n + 1 + 3) & ~3) +
                   ((lv.n_nbr + 3) & ~3);
        ints = std::max(ints, s);
    }
    const size_t xbuf = (size_t)kWarps * 4 * KF * sizeof(float);
    auto need = [&](int S, bool with_ints) {
        return (size_t)max_slots * S * kD * sizeof(float) + xbuf + (with_ints ? ints * sizeof(int) : 0);
    };
    p.ints_in_smem = 1;
    if (need(p.S, true) > budget) {
        if (need(p.S, false) <= budget) p.ints_in_smem = 0;
        else {
            // narrower slices (more blocks than half the SMs: they queue up)
            while (p.S > 1 && need(p.S, true) > budget) --p.S;
            if (need(p.S, true) > budget) p.ints_in_smem = 0;
            if (need(p.S, p.ints_in_smem != 0) > budget) return cudaErrorNotSupported;
        }
    }
    p.n_slices = (a.B + p.S - 1) / p.S;
    p.smem_bytes = need(p.S, p.ints_in_smem != 0);
    void (*kern)(const EmbedArgs, const D32Plan) = nullptr;
    switch (F4) {
        case 1: kern = embed_d32_kernel<1>; break;
        case 2: kern = embed_d32_kernel<2>; break;
        case 3: kern = embed_d32_kernel<3>; break;
        case 4: kern = embed_d32_kernel<4>; break;
        default: return cudaErrorNotSupported;
    }
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)p.smem_bytes);
    if (err != cudaSuccess) return err;
    kern<<<dim3(p.n_slices, 2), kThreads, p.smem_bytes, stream>>>(a, p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace placeto
