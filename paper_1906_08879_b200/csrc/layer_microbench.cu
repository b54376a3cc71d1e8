// Stand-alone microbenchmark (not part of libplaceto.so) of the building block of
// the d = 32 message-passing kernel: one 32 -> 32 layer for R rows per warp with
// the weights in registers and the activations exchanged through shared memory
// (store, warp barrier, eight broadcast 128-bit loads, 32 FMAs, ReLU), plus the
// primitive latencies it is made of. It reports cycles per layer for one warp
// alone (the latency floor of a level's dependent chain) and for 4 and 8 warps
// (the throughput ceiling of a wide level).
//
//   nvcc -O3 -std=c++17 -gencode arch=compute_100a,code=sm_100a \
//        -o layer_microbench paper_1906_08879_b200/csrc/layer_microbench.cu && ./layer_microbench
#include <cstdio>
#include <cuda_runtime.h>

typedef unsigned long long u64;

constexpr int kIters = 256;
constexpr int kMaxWarps = 8;      // blocks are launched with at most 8 warps

__device__ __forceinline__ unsigned clk() {
    unsigned t;
    asm volatile("mov.u32 %0, %%clock;" : "=r"(t)::"memory");
    return t;
}
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 pack(float lo, float hi) {
    u64 d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack(u64 v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

// ---- primitive latencies (one warp, dependent chains) ----
__global__ void k_fma(float *out, unsigned *t, float a, float b) {
    float x = out[threadIdx.x];
    const unsigned t0 = clk();
#pragma unroll
    for (int i = 0; i < kIters; ++i) x = fmaf(x, a, b);
    const unsigned t1 = clk();
    out[threadIdx.x] = x;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}
__global__ void k_lds128(float *out, unsigned *t) {   // dependent broadcast 128-bit loads
    __shared__ __align__(16) int4 s[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s[i] = make_int4((i + 1) & 255, 0, 0, 0);
    __syncthreads();
    int p = 0, acc = 0;
    const unsigned t0 = clk();
#pragma unroll
    for (int i = 0; i < kIters; ++i) {
        const int4 v = s[p];
        p = v.x;
        acc += v.y + v.z + v.w;
    }
    const unsigned t1 = clk();
    out[threadIdx.x] = (float)(p + acc);
    if (threadIdx.x == 0) t[0] = t1 - t0;
}
__global__ void k_exchange(float *out, unsigned *t) {   // store -> warp barrier -> load of another lane's value
    __shared__ float s[32];
    float x = out[threadIdx.x];
    const int lane = threadIdx.x & 31;
    const unsigned t0 = clk();
#pragma unroll
    for (int i = 0; i < kIters; ++i) {
        s[lane] = x;
        __syncwarp();
        x = s[(lane + 1) & 31] + 1.f;
        __syncwarp();
    }
    const unsigned t1 = clk();
    out[threadIdx.x] = x;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}
__global__ void k_shfl(float *out, unsigned *t) {
    float x = out[threadIdx.x];
    const unsigned t0 = clk();
#pragma unroll
    for (int i = 0; i < kIters; ++i) x = __shfl_xor_sync(0xffffffffu, x, 16) + 1.f;
    const unsigned t1 = clk();
    out[threadIdx.x] = x;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}
__global__ void k_barrier(float *out, unsigned *t) {
    const unsigned t0 = clk();
#pragma unroll 1
    for (int i = 0; i < kIters; ++i) __syncthreads();
    const unsigned t1 = clk();
    if (threadIdx.x == 0) { t[0] = t1 - t0; out[0] = 0.f; }
}

// ---- the layer: R rows per warp, NA accumulators per row ----
template <int R, int NA>
__global__ void k_layer(float *out, unsigned *t, const float *wsrc) {
    __shared__ __align__(16) float s[kMaxWarps][R * 32];
    const int lane = threadIdx.x & 31, warp = (threadIdx.x >> 5) % kMaxWarps;
    float w[32];
#pragma unroll
    for (int k = 0; k < 32; ++k) w[k] = wsrc[k * 32 + lane];
    float x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = out[threadIdx.x] + r;
    float *buf = s[warp];
    const unsigned t0 = clk();
#pragma unroll 1
    for (int i = 0; i < kIters; ++i) {
#pragma unroll
        for (int r = 0; r < R; ++r) buf[r * 32 + lane] = x[r];
        __syncwarp();
        float a[R][NA];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int j = 0; j < NA; ++j) a[r][j] = j == 0 ? 0.1f : 0.f;
#pragma unroll
        for (int k = 0; k < 32; k += 4)
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float4 u = *reinterpret_cast<const float4 *>(buf + r * 32 + k);
                a[r][0 % NA] = fmaf(u.x, w[k], a[r][0 % NA]);
                a[r][1 % NA] = fmaf(u.y, w[k + 1], a[r][1 % NA]);
                a[r][2 % NA] = fmaf(u.z, w[k + 2], a[r][2 % NA]);
                a[r][3 % NA] = fmaf(u.w, w[k + 3], a[r][3 % NA]);
            }
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
            for (int st = NA / 2; st >= 1; st >>= 1)
#pragma unroll
                for (int j = 0; j < st; ++j) a[r][j] += a[r][j + st];
            x[r] = fmaxf(a[r][0], 0.f);
        }
        __syncwarp();
    }
    const unsigned t1 = clk();
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) sum += x[r];
    out[threadIdx.x] = sum;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}

// the same on packed FP32 pairs (fma.rn.f32x2): half the FMA issue slots
template <int R>
__global__ void k_layer_packed(float *out, unsigned *t, const float *wsrc) {
    __shared__ __align__(16) float s[kMaxWarps][R * 32];
    const int lane = threadIdx.x & 31, warp = (threadIdx.x >> 5) % kMaxWarps;
    u64 w[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) w[k] = pack(wsrc[(2 * k) * 32 + lane], wsrc[(2 * k + 1) * 32 + lane]);
    float x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = out[threadIdx.x] + r;
    float *buf = s[warp];
    const unsigned t0 = clk();
#pragma unroll 1
    for (int i = 0; i < kIters; ++i) {
#pragma unroll
        for (int r = 0; r < R; ++r) buf[r * 32 + lane] = x[r];
        __syncwarp();
        u64 a[R][2];
#pragma unroll
        for (int r = 0; r < R; ++r) { a[r][0] = pack(0.1f, 0.f); a[r][1] = 0ull; }
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const ulonglong2 u = *reinterpret_cast<const ulonglong2 *>(buf + r * 32 + 4 * k);
                a[r][0] = ffma2(u.x, w[2 * k], a[r][0]);
                a[r][1] = ffma2(u.y, w[2 * k + 1], a[r][1]);
            }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float l0, h0, l1, h1;
            unpack(a[r][0], l0, h0);
            unpack(a[r][1], l1, h1);
            x[r] = fmaxf((l0 + h0) + (l1 + h1), 0.f);
        }
        __syncwarp();
    }
    const unsigned t1 = clk();
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) sum += x[r];
    out[threadIdx.x] = sum;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}

// the layer split over half-warps: lane (half, c) holds rows [16 half, 16 half + 16)
// of columns c and c + 16, reads half of the input and trades one partial sum
template <int R>
__global__ void k_layer_split(float *out, unsigned *t, const float *wsrc) {
    __shared__ __align__(16) float s[kMaxWarps][R * 32];
    const int lane = threadIdx.x & 31, warp = (threadIdx.x >> 5) % kMaxWarps;
    const int half = lane >> 4, col = lane & 15;
    float wa[16], wb[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        wa[k] = wsrc[(16 * half + k) * 32 + col];
        wb[k] = wsrc[(16 * half + k) * 32 + col + 16];
    }
    float x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = out[threadIdx.x] + r;
    float *buf = s[warp];
    const unsigned t0 = clk();
#pragma unroll 1
    for (int i = 0; i < kIters; ++i) {
#pragma unroll
        for (int r = 0; r < R; ++r) buf[r * 32 + lane] = x[r];
        __syncwarp();
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float p0 = half ? 0.f : 0.1f, p1 = half ? 0.1f : 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll
            for (int k = 0; k < 16; k += 4) {
                const float4 u = *reinterpret_cast<const float4 *>(buf + r * 32 + 16 * half + k);
                p0 = fmaf(u.x, wa[k], p0); p1 = fmaf(u.x, wb[k], p1);
                q0 = fmaf(u.y, wa[k + 1], q0); q1 = fmaf(u.y, wb[k + 1], q1);
                p0 = fmaf(u.z, wa[k + 2], p0); p1 = fmaf(u.z, wb[k + 2], p1);
                q0 = fmaf(u.w, wa[k + 3], q0); q1 = fmaf(u.w, wb[k + 3], q1);
            }
            const float c0 = p0 + q0, c1 = p1 + q1;
            const float send = half ? c0 : c1, keep = half ? c1 : c0;
            x[r] = fmaxf(keep + __shfl_xor_sync(0xffffffffu, send, 16), 0.f);
        }
        __syncwarp();
    }
    const unsigned t1 = clk();
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) sum += x[r];
    out[threadIdx.x] = sum;
    if (threadIdx.x == 0) t[0] = t1 - t0;
}

// Throughput of 128-bit shared loads by address pattern: eight warps each issue
// kIters x 16 loads whose 16-byte chunks are spread over the lanes as `pattern`
// says (no bank conflicts in any of them); reports cycles per load per SM. The
// loads are volatile so that none is merged or hoisted.
__global__ void __launch_bounds__(256) k_lds_pattern(float *out, unsigned *t, int pattern) {
    __shared__ __align__(16) float buf[8192];
    for (int i = threadIdx.x; i < 8192; i += blockDim.x) buf[i] = (float)i;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int off;   // float offset of this lane's chunk
    switch (pattern) {
        case 0: off = 0; break;                    // one address for the warp
        case 1: off = (lane >> 4) * 36; break;     // one per half-warp
        case 2: off = (lane >> 3) * 36; break;     // one per quarter-warp (8 consecutive lanes)
        case 3: off = (lane >> 2) * 76; break;     // one per group of 4 lanes: 2 per quarter-warp
        case 4: off = (lane & 1) * 36; break;      // 2 addresses alternating by lane
        case 5: off = (lane & 3) * 36; break;      // 4 addresses by lane mod 4: 4 per quarter-warp
        case 6: off = (lane & 7) * 4; break;       // 8 adjacent chunks, the same in every quarter-warp
        default: off = lane * 4; break;            // 32 distinct adjacent chunks
    }
    const unsigned base = (unsigned)__cvta_generic_to_shared(buf + off + warp * 4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    const unsigned t0 = clk();
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            float4 v;
            asm volatile("ld.volatile.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                         : "r"(base + (unsigned)(u % 8) * 256u));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    const unsigned t1 = clk();
    __syncthreads();
    if (threadIdx.x == 0) *t = t1 - t0;
    out[threadIdx.x] = acc.x + acc.y + acc.z + acc.w;
}

int main() {
    float *out, *w;
    unsigned *t, h = 0;
    if (cudaMalloc(&out, 8192) != cudaSuccess || cudaMalloc(&t, 64) != cudaSuccess ||
        cudaMalloc(&w, 4096) != cudaSuccess) {
        printf("no CUDA device\n");
        return 1;
    }
    cudaMemset(out, 0, 8192);
    {
        float hw[1024];
        for (int i = 0; i < 1024; ++i) hw[i] = 0.01f * ((i * 37) % 17 - 8);
        cudaMemcpy(w, hw, 4096, cudaMemcpyHostToDevice);
    }
#define PRIM(name, call)                                                          \
    for (int rep = 0; rep < 2; ++rep) {                                           \
        call;                                                                     \
        cudaDeviceSynchronize();                                                  \
        cudaMemcpy(&h, t, 4, cudaMemcpyDeviceToHost);                             \
    }                                                                             \
    printf("%-44s %6.1f cycles  (%s)\n", name, h / (double)kIters, cudaGetErrorString(cudaGetLastError()));
    PRIM("dependent FMA", (k_fma<<<1, 32>>>(out, t, 1.0001f, 0.5f)))
    PRIM("dependent broadcast 128-bit shared load", (k_lds128<<<1, 32>>>(out, t)))
    PRIM("shared store -> warp barrier -> load", (k_exchange<<<1, 32>>>(out, t)))
    PRIM("shuffle + add", (k_shfl<<<1, 32>>>(out, t)))
    PRIM("__syncthreads, 8 warps", (k_barrier<<<1, 256>>>(out, t)))
#define LAYER(name, kern, R)                                                                         \
    for (int warps : {1, 4, 8}) {                                                                    \
        for (int rep = 0; rep < 2; ++rep) {                                                          \
            kern<<<1, 32 * warps>>>(out, t, w);                                                      \
            cudaDeviceSynchronize();                                                                 \
            cudaMemcpy(&h, t, 4, cudaMemcpyDeviceToHost);                                            \
        }                                                                                            \
        printf("%-30s R=%d warps=%d  %6.1f cycles/layer  %5.1f cycles per row-layer per SM  (%s)\n", \
               name, R, warps, h / (double)kIters, h / (double)kIters / (R * warps),                 \
               cudaGetErrorString(cudaGetLastError()));                                              \
    }
    LAYER("fma, 1 accumulator", (k_layer<1, 1>), 1)
    LAYER("fma, 2 accumulators", (k_layer<1, 2>), 1)
    LAYER("fma, 4 accumulators", (k_layer<1, 4>), 1)
    LAYER("packed fma (f32x2)", (k_layer_packed<1>), 1)
    LAYER("half-warp split", (k_layer_split<1>), 1)
    LAYER("fma, 2 accumulators", (k_layer<2, 2>), 2)
    LAYER("fma, 4 accumulators", (k_layer<2, 4>), 2)
    LAYER("packed fma (f32x2)", (k_layer_packed<2>), 2)
    LAYER("half-warp split", (k_layer_split<2>), 2)
    LAYER("fma, 2 accumulators", (k_layer<4, 2>), 4)
    const char *patterns[] = {"one address per warp", "one per half-warp", "one per quarter-warp",
                              "one per 4 lanes (2 per quarter-warp)", "2 alternating by lane",
                              "4 by lane mod 4 (4 per quarter-warp)", "8 adjacent chunks per quarter-warp",
                              "32 distinct chunks"};
    for (int pat = 0; pat < 8; ++pat) {
        for (int rep = 0; rep < 2; ++rep) {
            k_lds_pattern<<<1, 256>>>(out, t, pat);
            cudaDeviceSynchronize();
            cudaMemcpy(&h, t, 4, cudaMemcpyDeviceToHost);
        }
        printf("128-bit shared load, %-38s %5.2f cycles per load per SM, 8 warps  (%s)\n", patterns[pat],
               h / (double)kIters / (16 * 8), cudaGetErrorString(cudaGetLastError()));
    }
    cudaFree(out); cudaFree(t); cudaFree(w);
    return 0;
}
