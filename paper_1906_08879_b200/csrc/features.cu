// Step 1 of the policy (Sec. 2.1 and Sec. 2.2 step 1 of the Placeto paper):
// raw per-node, per-state features
//   x = [cost, bytes, one-hot(device), is-current, is-placed],  F = m + 4,
// written as X[n][B][F]. The state arrays are state-major (dev[B][n]) while X
// is node-major, so a block transposes a 32-node x 32-state tile through
// shared memory: loads run along nodes, stores along (state, feature).
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kTile = 32;

__global__ void __launch_bounds__(256)
features_kernel(int n, int B, int m, const float *__restrict__ cost,
                const float *__restrict__ bytes, const uint8_t *__restrict__ dev,
                const int *__restrict__ cur, const uint8_t *__restrict__ placed,
                float *__restrict__ X) {
    dependents_may_start();
    __shared__ uint8_t s_dev[kTile][kTile + 4];
    __shared__ uint8_t s_placed[kTile][kTile + 4];
    __shared__ int s_cur[kTile];
    __shared__ float s_cost[kTile], s_bytes[kTile];
    const int v0 = blockIdx.x * kTile, b0 = blockIdx.y * kTile;
    const int F = m + 4;
    dependency_wait();          // the inputs may come from the gather kernel of the same call
    for (int i = threadIdx.x; i < kTile * kTile; i += blockDim.x) {
        const int bl = i / kTile, vl = i % kTile;
        const int b = b0 + bl, v = v0 + vl;
        const bool ok = b < B && v < n;
        s_dev[bl][vl] = ok ? dev[(size_t)b * n + v] : 0;
        s_placed[bl][vl] = ok ? placed[(size_t)b * n + v] : 0;
    }
    if (threadIdx.x < kTile) s_cur[threadIdx.x] = (b0 + threadIdx.x < B) ? cur[b0 + threadIdx.x] : -1;
    if (threadIdx.x >= 32 && threadIdx.x < 32 + kTile && v0 + threadIdx.x - 32 < n) {
        s_cost[threadIdx.x - 32] = cost[v0 + threadIdx.x - 32];
        s_bytes[threadIdx.x - 32] = bytes[v0 + threadIdx.x - 32];
    }
    __syncthreads();
    const int nb = min(kTile, B - b0);
    const int nv = min(kTile, n - v0);
    // one (node, state) pair per thread pass: its F features are contiguous in X,
    // and the pairs of one node follow each other, so a warp writes 32 F floats in a row
    for (int i = threadIdx.x; i < nv * kTile; i += blockDim.x) {
        const int vl = i / kTile, bl = i % kTile;
        if (bl >= nb) continue;
        const int v = v0 + vl;
        float *out = X + ((size_t)v * B + b0 + bl) * F;
        const int d = s_dev[bl][vl];
        const float cur_flag = (s_cur[bl] == v) ? 1.f : 0.f;
        const float placed_flag = s_placed[bl][vl] ? 1.f : 0.f;
        if ((F & 3) == 0) {
            for (int k = 0; k < F; k += 4) {
                float t[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int kk = k + j;
                    t[j] = kk == 0 ? s_cost[vl] : kk == 1 ? s_bytes[vl]
                         : kk < 2 + m ? (d == kk - 2 ? 1.f : 0.f)
                         : kk == 2 + m ? cur_flag : placed_flag;
                }
                *reinterpret_cast<float4 *>(out + k) = make_float4(t[0], t[1], t[2], t[3]);
            }
        } else {
            for (int kk = 0; kk < F; ++kk)
                out[kk] = kk == 0 ? s_cost[vl] : kk == 1 ? s_bytes[vl]
                        : kk < 2 + m ? (d == kk - 2 ? 1.f : 0.f)
                        : kk == 2 + m ? cur_flag : placed_flag;
        }
    }
}

// Gathers the host-resident inputs of one policy evaluation into device memory
// in a single launch. The sources are page-locked host buffers that the device
// can address; a warp reads 512 contiguous bytes per pass (16 bytes per lane), so
// the reads cross the host link as full-size requests.
struct StageSegments {
    const char *src[5];
    char *dst[5];
    size_t bytes[5];
};

__global__ void __launch_bounds__(256)
stage_inputs_kernel(const StageSegments s) {
    dependents_may_start();
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const char *src = s.src[i];
        char *dst = s.dst[i];
        const size_t bytes = s.bytes[i];
        size_t done = 0;
        if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0) {
            const size_t words = bytes / 16;
            for (size_t k = tid; k < words; k += stride)
                reinterpret_cast<uint4 *>(dst)[k] = reinterpret_cast<const uint4 *>(src)[k];
            done = words * 16;
        }
        for (size_t k = done + tid; k < bytes; k += stride) dst[k] = src[k];
    }
}

}  // namespace

cudaError_t launch_stage_inputs(const void *const (&src)[5], void *const (&dst)[5],
                                const size_t (&bytes)[5], int sm_count, cudaStream_t stream) {
    StageSegments s;
    size_t total = 0;
    for (int i = 0; i < 5; ++i) {
        s.src[i] = static_cast<const char *>(src[i]);
        s.dst[i] = static_cast<char *>(dst[i]);
        s.bytes[i] = bytes[i];
        total += bytes[i];
    }
    // one 16-byte word per thread up to two blocks per SM, grid-stride beyond
    const size_t want = (total / 16 + 255) / 256 + 1;
    const int grid = (int)std::min<size_t>(want, (size_t)2 * sm_count);
    stage_inputs_kernel<<<grid, 256, 0, stream>>>(s);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_features(int n, int B, int m, const float *cost, const float *bytes,
                            const uint8_t *dev, const int *cur, const uint8_t *placed, float *X,
                            cudaStream_t stream, bool overlap) {
    dim3 grid((n + kTile - 1) / kTile, (B + kTile - 1) / kTile);
    cudaError_t err = launch_overlapped(overlap, features_kernel, grid, dim3(256), 0, stream, n, B, m, cost,
                                        bytes, dev, cur, placed, X);
    count_launch();
    return err;
}

}  // namespace placeto
