// Gradient of the policy objective with respect to every weight (Appendix A.1
// and A.7 of the Placeto paper: the REINFORCE term sum_b A_b log pi(a_b | s_b)
// plus an entropy term beta sum_b H(pi(. | s_b))), by reverse-mode
// differentiation of the forward path:
//
//   1. messages   : for every (node, state) row the hidden layer and the output of
//                   f are recomputed from H and X and stored (both directions);
//   2. head/pool  : per state, the pooled sums, h_i, the head and the softmax are
//                   recomputed, d(objective)/d(logits) is formed and pushed back
//                   through the head, h_i and l_i down to d/d(e_u) of every node;
//   3. sweeps     : per direction, levels in reverse order, d/d(h_v) is pushed
//                   through g to the summed messages and through f to the
//                   neighbours' embeddings (a node gathers from its consumers:
//                   no scattered adds);
//   4. weights    : each network layer's dW = in^T dpre and db = sum dpre over the
//                   stored per-row inputs and pre-activation gradients, as a
//                   chunked product with partials added in a fixed order.
// Nothing is accumulated with atomics: results are reproducible bit for bit.
// The kernels are dimension-generic (one thread per output element); shapes:
// two-layer ReLU f and g, single-layer ReLU l_i and h_i, two-layer head with a
// ReLU hidden layer and a linear output.
#include <algorithm>

#include "kernels.cuh"

namespace placeto {

namespace {

constexpr int kThreads = 256;
constexpr int kRows = 32;          // rows per pass of the row kernels

// ---------------------------------------------------------------- 1. messages
// FH = relu([H || X] W1 + b1), M = relu(FH W2 + b2) for all rows of one direction.
__global__ void __launch_bounds__(kThreads)
grad_messages_kernel(const GradArgs a) {
    extern __shared__ __align__(16) float smem[];
    const int dir = blockIdx.y;
    const DevMlp f = a.f[dir];
    const int d = a.d, F = a.F, Hf = f.hidden_dim, K = d + F;
    float *in = smem;                      // [kRows][K]
    float *hid = in + kRows * K;           // [kRows][Hf]
    const float *H = a.H[dir];
    const size_t R = (size_t)a.n * a.B;
    for (size_t r0 = (size_t)blockIdx.x * kRows; r0 < R; r0 += (size_t)gridDim.x * kRows) {
        const int rows = (int)min((size_t)kRows, R - r0);
        for (int i = threadIdx.x; i < rows * K; i += kThreads) {
            const int r = i / K, k = i - r * K;
            in[i] = k < d ? H[(r0 + r) * d + k] : a.X[(r0 + r) * F + (k - d)];
        }
        __syncthreads();
        for (int i = threadIdx.x; i < rows * Hf; i += kThreads) {
            const int r = i / Hf, j = i - r * Hf;
            float acc = f.b1[j];
            for (int k = 0; k < K; ++k) acc = fmaf(in[r * K + k], f.W1[k * Hf + j], acc);
            acc = fmaxf(acc, 0.f);
            hid[i] = acc;
            a.FH[dir][(r0 + r) * Hf + j] = acc;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < rows * d; i += kThreads) {
            const int r = i / d, j = i - r * d;
            float acc = f.b2[j];
            for (int k = 0; k < Hf; ++k) acc = fmaf(hid[r * Hf + k], f.W2[k * d + j], acc);
            a.M[dir][(r0 + r) * d + j] = fmaxf(acc, 0.f);
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------- 2. head / pool
// One block per state (grid-stride). Shared memory: the state's vectors.
__global__ void __launch_bounds__(kThreads)
grad_head_kernel(const GradArgs a) {
    extern __shared__ __align__(16) float smem[];
    const int d = a.d, F = a.F, m = a.m, n = a.n, B = a.B;
    const int E = 2 * d + F, Z = 5 * d + F, Hh = a.head.hidden_dim;
    constexpr int G = kThreads / 32;       // nodes handled per iteration, one warp each
    float *z = smem;                       // [Z]
    float *hid = z + Z;                    // [Hh]
    float *dhid = hid + Hh;                // [Hh]
    float *dz = dhid + Hh;                 // [Z]
    float *S = dz + Z;                     // [3][d]
    float *dS = S + 3 * d;                 // [3][d]
    float *lg = dS + 3 * d;                // [m] logits, then d/d(logits)
    float *part = lg + ((m + 3) & ~3);     // [G][3][d] partial sums / [G][d] exchange
    float *erow = part + G * 3 * d;        // [G][E]: the embedding row a warp is working on
    float *wl = erow + G * ((E + 3) & ~3); // [3][E * d + d]: the three l_i (weights, then bias)
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int lsz = E * d + d;
    for (int i = 0; i < 3; ++i) {
        for (int t = threadIdx.x; t < E * d; t += kThreads) wl[i * lsz + t] = a.l[i].W1[t];
        for (int t = threadIdx.x; t < d; t += kThreads) wl[i * lsz + E * d + t] = a.l[i].b1[t];
    }
    float *my_e = erow + g * ((E + 3) & ~3);
    __syncthreads();
    for (int b = blockIdx.x; b < B; b += gridDim.x) {
        const int c = a.cur[b];
        if (c < 0 || c >= n) {             // no such node: the state contributes nothing
            for (int i = threadIdx.x; i < n * d; i += kThreads) {
                const size_t off = ((size_t)(i / d) * B + b) * d + (i % d);
                a.DH[0][off] = 0.f;
                a.DH[1][off] = 0.f;
            }
            for (int k = threadIdx.x; k < Z; k += kThreads) a.Zbuf[(size_t)b * Z + k] = 0.f;
            for (int k = threadIdx.x; k < Hh; k += kThreads) { a.HID[(size_t)b * Hh + k] = 0.f; a.DHID[(size_t)b * Hh + k] = 0.f; }
            for (int k = threadIdx.x; k < m; k += kThreads) a.DLOG[(size_t)b * m + k] = 0.f;
            for (int k = threadIdx.x; k < 3 * d; k += kThreads) { a.Sbuf[(size_t)b * 3 * d + k] = 0.f; a.DPRE_H[(size_t)b * 3 * d + k] = 0.f; }
            continue;
        }
        const uint8_t *rel = a.relation + (size_t)c * n;
        auto e_of = [&](int u, int k) -> float {
            return k < d ? a.H[0][((size_t)u * B + b) * d + k]
                 : k < 2 * d ? a.H[1][((size_t)u * B + b) * d + (k - d)]
                             : a.X[((size_t)u * B + b) * F + (k - 2 * d)];
        };
        // ---- pooled sums S_i = sum_{u in set i} relu(l_i(e_u)); warp g takes nodes g, g + G, ...
        for (int i = threadIdx.x; i < G * 3 * d; i += kThreads) part[i] = 0.f;
        __syncthreads();
        for (int u = g; u < n; u += G) {
            const int set = rel[u];
            if (set > 2) continue;
            const float *W = wl + set * lsz;
            __syncwarp();
            for (int k = lane; k < E; k += 32) my_e[k] = e_of(u, k);
            __syncwarp();
            for (int j = lane; j < d; j += 32) {
                float acc = W[E * d + j];
                for (int k = 0; k < E; ++k) acc = fmaf(my_e[k], W[k * d + j], acc);
                part[(g * 3 + set) * d + j] += fmaxf(acc, 0.f);
            }
        }
        __syncthreads();
        for (int i = threadIdx.x; i < 3 * d; i += kThreads) {
            float acc = 0.f;
            for (int q = 0; q < G; ++q) acc += part[q * 3 * d + i];
            S[i] = acc;
            a.Sbuf[(size_t)b * 3 * d + i] = acc;
        }
        for (int k = threadIdx.x; k < E; k += kThreads) z[k] = e_of(c, k);
        __syncthreads();
        // ---- a_i = relu(h_i(S_i)) into z, hidden layer, logits
        for (int i = threadIdx.x; i < 3 * d; i += kThreads) {
            const int set = i / d, j = i - set * d;
            const DevMlp &h = a.h[set];
            float acc = h.b1[j];
            for (int k = 0; k < d; ++k) acc = fmaf(S[set * d + k], h.W1[k * d + j], acc);
            z[E + i] = fmaxf(acc, 0.f);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < Hh; j += kThreads) {
            float acc = a.head.b1[j];
#pragma unroll 8
            for (int k = 0; k < Z; ++k) acc = fmaf(z[k], a.head.W1[(size_t)k * Hh + j], acc);
            hid[j] = fmaxf(acc, 0.f);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < m; j += kThreads) {
            float acc = a.head.b2[j];
            for (int k = 0; k < Hh; ++k) acc = fmaf(hid[k], a.head.W2[(size_t)k * m + j], acc);
            lg[j] = acc;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            // d/d(logit_k) of A log p[a] + beta H = A (1[k = a] - p_k) - beta p_k (log p_k + H)
            float mx = lg[0];
            for (int k = 1; k < m; ++k) mx = fmaxf(mx, lg[k]);
            float tot = 0.f;
            for (int k = 0; k < m; ++k) tot += expf(lg[k] - mx);
            const float lt = logf(tot);
            float ent = 0.f;
            for (int k = 0; k < m; ++k) {
                const float lp = lg[k] - mx - lt;
                ent -= expf(lp) * lp;
            }
            const float A = a.advantages[b];
            const int act = a.actions[b];
            for (int k = 0; k < m; ++k) {
                const float lp = lg[k] - mx - lt, p = expf(lp);
                lg[k] = A * ((k == act ? 1.f : 0.f) - p) - a.beta * p * (lp + ent);
            }
        }
        __syncthreads();
        for (int k = threadIdx.x; k < Z; k += kThreads) a.Zbuf[(size_t)b * Z + k] = z[k];
        for (int j = threadIdx.x; j < m; j += kThreads) a.DLOG[(size_t)b * m + j] = lg[j];
        for (int k = threadIdx.x; k < Hh; k += kThreads) {
            float acc = 0.f;
            for (int j = 0; j < m; ++j) acc = fmaf(lg[j], a.head.W2[(size_t)k * m + j], acc);
            acc = hid[k] > 0.f ? acc : 0.f;
            dhid[k] = acc;
            a.HID[(size_t)b * Hh + k] = hid[k];
            a.DHID[(size_t)b * Hh + k] = acc;
        }
        __syncthreads();
        for (int i = g; i < Z; i += G) {       // a warp per input: its weight row is contiguous
            float acc = 0.f;
            for (int k = lane; k < Hh; k += 32) acc = fmaf(dhid[k], a.head.W1[(size_t)i * Hh + k], acc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) dz[i] = acc;
        }
        __syncthreads();
        // through h_i: dpre_h = dz_a * (a > 0); dS = dpre_h W_h^T
        for (int i = threadIdx.x; i < 3 * d; i += kThreads) {
            const float v = z[E + i] > 0.f ? dz[E + i] : 0.f;
            part[i] = v;
            a.DPRE_H[(size_t)b * 3 * d + i] = v;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < 3 * d; i += kThreads) {
            const int set = i / d, k = i - set * d;
            const DevMlp &h = a.h[set];
            float acc = 0.f;
            for (int j = 0; j < d; ++j) acc = fmaf(part[set * d + j], h.W1[k * d + j], acc);
            dS[i] = acc;
        }
        __syncthreads();
        // ---- through l_i to every node: dpre_l = dS_set * (pre > 0); de = dpre_l W_l^T
        float *xch = part;                 // [G][d]
        for (int u0 = 0; u0 < n; u0 += G) {
            const int u = u0 + g;
            const int set = u < n ? rel[u] : 3;
            if (set <= 2) {
                const float *W = wl + set * lsz;
                for (int k = lane; k < E; k += 32) my_e[k] = e_of(u, k);
                __syncwarp();
                for (int j = lane; j < d; j += 32) {
                    float acc = W[E * d + j];
                    for (int k = 0; k < E; ++k) acc = fmaf(my_e[k], W[k * d + j], acc);
                    const float v = acc > 0.f ? dS[set * d + j] : 0.f;
                    xch[g * d + j] = v;
                    a.DPRE_L[set][((size_t)u * B + b) * d + j] = v;
                }
            }
            __syncwarp();
            if (set <= 2) {
                const float *W = wl + set * lsz;
                for (int k = lane; k < 2 * d; k += 32) {
                    float acc = 0.f;
                    for (int j = 0; j < d; ++j) {
                        const int jj = (j + lane) % d;     // rotated per lane: no shared-memory bank conflicts
                        acc = fmaf(xch[g * d + jj], W[k * d + jj], acc);
                    }
                    float *dst = k < d ? a.DH[0] : a.DH[1];
                    dst[((size_t)u * B + b) * d + (k < d ? k : k - d)] = acc;
                }
            } else if (u < n) {            // the current node: its embedding enters the head directly
                for (int k = lane; k < 2 * d; k += 32) {
                    float *dst = k < d ? a.DH[0] : a.DH[1];
                    dst[((size_t)u * B + b) * d + (k < d ? k : k - d)] = dz[k];
                }
            }
            __syncwarp();
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ 3. sweeps
constexpr int kSweepRows = 64;     // rows per pass of the sweep kernel

// out(r, j) = sum_k A[r][k] W[k][j] for rows x J outputs, all operands in shared
// memory (A row stride lda, odd; W row stride ldw, a multiple of 4). A thread owns
// tiles of 2 rows x 4 columns: two scalar loads and one 128-bit load feed 8 FMAs.
template <typename Epilogue>
__device__ __forceinline__ void tile_product(const float *A, int lda, const float *W, int ldw, int K,
                                             int J, int rows, Epilogue done) {
    if (rows * J <= 2 * kThreads) {
        // a short pass (narrow level, few states): one output per thread keeps the chain short
        for (int i = threadIdx.x; i < rows * J; i += kThreads) {
            const int r = i / J, j = i - r * J;
            const float *x = A + r * lda, *w = W + j;
            float c = 0.f, e = 0.f;
            int k = 0;
            for (; k + 2 <= K; k += 2) {
                c = fmaf(x[k], w[k * ldw], c);
                e = fmaf(x[k + 1], w[(k + 1) * ldw], e);
            }
            if (k < K) c = fmaf(x[k], w[k * ldw], c);
            done(r, j, c + e);
        }
        return;
    }
    const int tiles_j = (J + 3) >> 2, tiles_r = (rows + 1) >> 1;
    for (int tile = threadIdx.x; tile < tiles_r * tiles_j; tile += kThreads) {
        const int tr = tile / tiles_j, tj = tile - tr * tiles_j;
        const int r0 = 2 * tr, r1 = min(r0 + 1, rows - 1);
        const float *a0 = A + r0 * lda, *a1 = A + r1 * lda, *w = W + 4 * tj;
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        for (int k = 0; k < K; ++k) {
            const float4 wv = *reinterpret_cast<const float4 *>(w + k * ldw);
            const float x0 = a0[k], x1 = a1[k];
            c0[0] = fmaf(x0, wv.x, c0[0]); c0[1] = fmaf(x0, wv.y, c0[1]);
            c0[2] = fmaf(x0, wv.z, c0[2]); c0[3] = fmaf(x0, wv.w, c0[3]);
            c1[0] = fmaf(x1, wv.x, c1[0]); c1[1] = fmaf(x1, wv.y, c1[1]);
            c1[2] = fmaf(x1, wv.z, c1[2]); c1[3] = fmaf(x1, wv.w, c1[3]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = 4 * tj + q;
            if (j < J) {
                done(r0, j, c0[q]);
                if (r0 + 1 < rows) done(r0 + 1, j, c1[q]);
            }
        }
    }
}

// One block per (state slice, direction): levels in reverse order. Per pass of up
// to kSweepRows rows: one phase brings everything the pass needs from global
// memory into shared memory (so a level pays one memory latency, not one per
// step), then four shared-memory products push the gradient through f and g.
__global__ void __launch_bounds__(kThreads)
grad_sweep_kernel(const GradArgs a, int S) {
    extern __shared__ __align__(16) float smem[];
    const int dir = blockIdx.y;
    const DevLevels lv = a.lv[dir];
    const DevMlp f = a.f[dir], gm = a.g[dir];
    const int d = a.d, B = a.B, Hf = f.hidden_dim, Hg = gm.hidden_dim;
    const int b0 = blockIdx.x * S, nb = min(S, B - b0);
    // consumers of a node's message: children for the top-down pass, parents for the bottom-up one
    const int *cons_ptr = dir == 0 ? a.child_ptr : a.parent_ptr;
    const int *cons = dir == 0 ? a.child : a.parent;
    const int W = max(max(d, Hf), Hg) | 1;         // odd row stride of the row buffers
    float *bufA = smem;                            // [rows][W] dpre_f2, later dt1
    float *bufB = bufA + kSweepRows * W;           // dfh
    float *bufC = bufB + kSweepRows * W;           // dpre_g2
    float *bufD = bufC + kSweepRows * W;           // d/dh from the pooling
    float *bufS = bufD + kSweepRows * W;           // summed neighbour messages
    float *mskF = bufS + kSweepRows * W;           // fh > 0
    float *mskH = mskF + kSweepRows * W;           // h > 0
    // the direction's matrices, each in the orientation its product reads row-wise
    const int pd = (d + 3) & ~3, pf = (Hf + 3) & ~3, pg = (Hg + 3) & ~3;
    float *wf2t = mskH + kSweepRows * W;           // [d][pf]:  W_f2^T
    float *wf1t = wf2t + d * pf;                   // [Hf][pd]: (h rows of W_f1)^T
    float *wg1 = wf1t + Hf * pd;                   // [d][pg]:  W_g1
    float *wg2t = wg1 + d * pg;                    // [d][pg]:  W_g2^T
    float *wg1t = wg2t + d * pg;                   // [Hg][pd]: W_g1^T
    float *bg1 = wg1t + Hg * pd;                   // [Hg]
    for (int i = threadIdx.x; i < Hf * d; i += kThreads) { const int k = i / d, j = i - k * d; wf2t[j * pf + k] = f.W2[i]; }
    for (int i = threadIdx.x; i < d * Hf; i += kThreads) { const int j = i / Hf, k = i - j * Hf; wf1t[k * pd + j] = f.W1[i]; }
    for (int i = threadIdx.x; i < d * Hg; i += kThreads) { const int j = i / Hg, k = i - j * Hg; wg1[j * pg + k] = gm.W1[i]; wg1t[k * pd + j] = gm.W1[i]; }
    for (int i = threadIdx.x; i < Hg * d; i += kThreads) { const int k = i / d, j = i - k * d; wg2t[j * pg + k] = gm.W2[i]; }
    for (int i = threadIdx.x; i < Hg; i += kThreads) bg1[i] = gm.b1[i];
    __syncthreads();
    const float *H = a.H[dir], *M = a.M[dir], *FH = a.FH[dir];
    for (int level = lv.n_levels - 1; level >= 0; --level) {
        const int p0 = lv.level_ptr[level], width = lv.level_ptr[level + 1] - p0;
        const int total = width * nb;
        for (int r0 = 0; r0 < total; r0 += kSweepRows) {
            const int rows = min(kSweepRows, total - r0);
            auto row_of = [&](int r, int &pos, size_t &off) {
                const int q = (r0 + r) / nb;
                pos = p0 + q;
                off = (size_t)lv.order[pos] * B + b0 + (r0 + r - q * nb);
            };
            // ---- everything the pass reads from global memory
            for (int i = threadIdx.x; i < rows * d; i += kThreads) {
                const int r = i / d, j = i - r * d;
                int pos; size_t off;
                row_of(r, pos, off);
                const int u = lv.order[pos];
                const int b = (int)(off - (size_t)u * B);
                float dm = 0.f, s = 0.f;
                for (int e = cons_ptr[u]; e < cons_ptr[u + 1]; ++e)
                    dm += a.DS[dir][((size_t)cons[e] * B + b) * d + j];
                for (int e = lv.nbr_ptr[pos]; e < lv.nbr_ptr[pos + 1]; ++e)
                    s += M[((size_t)lv.nbr[e] * B + b) * d + j];
                dm = M[off * d + j] > 0.f ? dm : 0.f;            // dpre_f2
                bufA[r * W + j] = dm;
                a.DPRE_F2[dir][off * d + j] = dm;
                bufS[r * W + j] = s;
                a.Sg[dir][off * d + j] = s;
                bufD[r * W + j] = a.DH[dir][off * d + j];
                mskH[r * W + j] = H[off * d + j] > 0.f ? 1.f : 0.f;
            }
            for (int i = threadIdx.x; i < rows * Hf; i += kThreads) {
                const int r = i / Hf, k = i - r * Hf;
                int pos; size_t off;
                row_of(r, pos, off);
                mskF[r * W + k] = FH[off * Hf + k] > 0.f ? 1.f : 0.f;
            }
            __syncthreads();
            // ---- dfh = (dpre_f2 W_f2^T) * (fh > 0)
            tile_product(bufA, W, wf2t, pf, d, Hf, rows, [&](int r, int k, float v) {
                int pos; size_t off;
                row_of(r, pos, off);
                v *= mskF[r * W + k];
                bufB[r * W + k] = v;
                a.DFH[dir][off * Hf + k] = v;
            });
            __syncthreads();
            // ---- dpre_g2 = (dH_pool + dfh W_f1[0:d]^T) * (h > 0)
            tile_product(bufB, W, wf1t, pd, Hf, d, rows, [&](int r, int j, float v) {
                int pos; size_t off;
                row_of(r, pos, off);
                v = (v + bufD[r * W + j]) * mskH[r * W + j];
                bufC[r * W + j] = v;
                a.DPRE_G2[dir][off * d + j] = v;
            });
            __syncthreads();
            // ---- t1 = relu(s W_g1 + b), dt1 = (dpre_g2 W_g2^T) * (t1 > 0): t1 first, into bufA as a mask
            tile_product(bufS, W, wg1, pg, d, Hg, rows, [&](int r, int k, float v) {
                int pos; size_t off;
                row_of(r, pos, off);
                v = fmaxf(v + bg1[k], 0.f);
                a.T1[dir][off * Hg + k] = v;
                bufA[r * W + k] = v > 0.f ? 1.f : 0.f;
            });
            __syncthreads();
            tile_product(bufC, W, wg2t, pg, d, Hg, rows, [&](int r, int k, float v) {
                int pos; size_t off;
                row_of(r, pos, off);
                v *= bufA[r * W + k];
                a.DT1[dir][off * Hg + k] = v;
                bufB[r * W + k] = v;
            });
            __syncthreads();
            // ---- ds = dt1 W_g1^T
            tile_product(bufB, W, wg1t, pd, Hg, d, rows, [&](int r, int j, float v) {
                int pos; size_t off;
                row_of(r, pos, off);
                a.DS[dir][off * d + j] = v;
            });
            __syncthreads();
        }
        __threadfence_block();
        __syncthreads();               // the next (lower) level gathers this level's ds
    }
}

// ----------------------------------------------------------------- 4. weights
// partial[chunk][K][J] = sum over the chunk's rows of in[r][k] dp[r][j]; the input
// row is the concatenation of up to three arrays. Bias: partial_b[chunk][J].
struct WeightJob {
    const float *in[3];
    int width[3], stride[3];     // columns taken from each part, and its row stride
    const float *dp;
    int dp_stride;
    int K, J;
    size_t R;
    float *partial;       // [chunks][(K + 1) * J], row K holds the bias sums
    float *dW, *db;
    int chunks;
    int accumulate;       // 1: add to what dW, db hold instead of overwriting
};

constexpr int kMaxJobs = 16;
struct WeightJobs {
    WeightJob job[kMaxJobs];
    int count;
};

// All layers in one launch: blockIdx.z picks the job, blocks beyond a job's
// chunks or output tiles leave at once.
__global__ void __launch_bounds__(kThreads)
grad_weight_partial_kernel(const WeightJobs jobs) {
    extern __shared__ __align__(16) float smem[];
    const WeightJob &w = jobs.job[blockIdx.z];
    const int K = w.K, J = w.J;
    const int Kp = (K + 1 + 3) & ~3, Jp = (J + 3) & ~3;      // padded with zeros to whole 4 x 4 tiles
    const int tiles_j = Jp >> 2, n_tiles = (Kp >> 2) * tiles_j;
    if ((int)blockIdx.x >= w.chunks || (int)blockIdx.y * kThreads >= n_tiles) return;
    float *in = smem;                  // [kRows][Kp] (column K = 1 for the bias)
    float *dp = in + kRows * Kp;       // [kRows][Jp]
    const int chunk = blockIdx.x;
    const size_t per = (w.R + w.chunks - 1) / w.chunks;
    const size_t r_begin = (size_t)chunk * per, r_end = min(w.R, r_begin + per);
    // a thread owns one 4 x 4 tile of the product: two 128-bit shared loads feed 16 FMAs
    const int tile = blockIdx.y * kThreads + threadIdx.x;
    const bool live = tile < n_tiles;
    const int tk = live ? tile / tiles_j : 0, tj = live ? tile - tk * tiles_j : 0;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (size_t r0 = r_begin; r0 < r_end; r0 += kRows) {
        const int rows = (int)min((size_t)kRows, r_end - r0);
        for (int i = threadIdx.x; i < rows * Kp; i += kThreads) {
            const int r = i / Kp, k = i - r * Kp;
            float v = k == K ? 1.f : 0.f;
            if (k < K) {
                int kk = k, part = 0;
                while (kk >= w.width[part]) { kk -= w.width[part]; ++part; }
                v = w.in[part][(r0 + r) * w.stride[part] + kk];
            }
            in[i] = v;
        }
        for (int i = threadIdx.x; i < rows * Jp; i += kThreads) {
            const int r = i / Jp, j = i - r * Jp;
            dp[i] = j < J ? w.dp[(r0 + r) * w.dp_stride + j] : 0.f;
        }
        __syncthreads();
        if (live) {
            const float *pa = in + 4 * tk, *pb = dp + 4 * tj;
            for (int r = 0; r < rows; ++r) {
                const float4 x = *reinterpret_cast<const float4 *>(pa + r * Kp);
                const float4 y = *reinterpret_cast<const float4 *>(pb + r * Jp);
                const float xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xs[i], ys[j], acc[i][j]);
            }
        }
        __syncthreads();
    }
    if (live) {
        const int n_out = (K + 1) * J;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int k = 4 * tk + i, jj = 4 * tj + j;
                if (k <= K && jj < J) w.partial[(size_t)chunk * n_out + k * J + jj] = acc[i][j];
            }
    }
}

// Adds the chunk partials: a block owns 32 outputs; eight thread groups each add
// every eighth chunk (ascending), then the eight sums are added in group order.
__global__ void __launch_bounds__(256)
grad_weight_reduce_kernel(const WeightJobs jobs) {
    __shared__ float sums[8][32];
    const WeightJob &w = jobs.job[blockIdx.y];
    const int n_out = (w.K + 1) * w.J;
    if ((int)blockIdx.x * 32 >= n_out) return;
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int o = blockIdx.x * 32 + lane;
    float acc = 0.f;
    if (o < n_out)
        for (int c = grp; c < w.chunks; c += 8) acc += w.partial[(size_t)c * n_out + o];
    sums[grp][lane] = acc;
    __syncthreads();
    if (grp == 0 && o < n_out) {
        float total = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) total += sums[q][lane];
        float *dst = o < w.K * w.J ? w.dW + o : w.db + (o - w.K * w.J);
        *dst = w.accumulate ? *dst + total : total;
    }
}

cudaError_t weight_grads(const WeightJobs &jobs, cudaStream_t stream) {
    if (jobs.count == 0) return cudaSuccess;
    size_t smem = 0;
    int max_chunks = 1, max_out = 1, max_tiles = 1;
    for (int i = 0; i < jobs.count; ++i) {
        const WeightJob &w = jobs.job[i];
        const int Kp = (w.K + 1 + 3) & ~3, Jp = (w.J + 3) & ~3;
        smem = std::max(smem, (size_t)kRows * (Kp + Jp) * sizeof(float));
        max_chunks = std::max(max_chunks, w.chunks);
        max_out = std::max(max_out, (w.K + 1) * w.J);
        max_tiles = std::max(max_tiles, (Kp / 4) * (Jp / 4));
    }
    cudaError_t err = cudaFuncSetAttribute(grad_weight_partial_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    grad_weight_partial_kernel<<<dim3(max_chunks, (max_tiles + kThreads - 1) / kThreads, jobs.count), kThreads, smem, stream>>>(jobs);
    count_launch();
    grad_weight_reduce_kernel<<<dim3((max_out + 31) / 32, jobs.count), 256, 0, stream>>>(jobs);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

namespace {
__global__ void identity_layer_kernel(float *dst, int d) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < d * d + d) dst[i] = (i < d * d && i / d == i % d) ? 1.f : 0.f;
}
}  // namespace

cudaError_t launch_identity_layer(float *dst, int d, cudaStream_t stream) {
    identity_layer_kernel<<<(d * d + d + 255) / 256, 256, 0, stream>>>(dst, d);
    count_launch();
    return cudaGetLastError();
}

bool policy_gradient_applicable(const GradArgs &a) {
    auto relu2 = [](const DevMlp &m) { return m.n_layers == 2 && m.act == 0 && m.final_act == 1; };
    auto relu1 = [](const DevMlp &m) { return m.n_layers == 1 && m.act == 0 && m.final_act == 1; };
    for (int dir = 0; dir < 2; ++dir)
        if (!relu2(a.f[dir]) || !relu2(a.g[dir])) return false;
    for (int i = 0; i < 3; ++i)
        if (!relu1(a.l[i]) || !relu1(a.h[i])) return false;
    return a.head.n_layers == 2 && a.head.act == 0 && a.head.final_act == 0;
}

// floats of workspace (every array padded to a multiple of 4 floats by the carve below)
size_t policy_gradient_workspace_floats(int n, int B, int d, int F, int m, int Hf, int Hg, int Hh) {
    const size_t R = (size_t)n * B, Z = 5 * (size_t)d + F, E = 2 * (size_t)d + F;
    const size_t per_dir = R * ((size_t)Hf * 2 + (size_t)Hg * 2 + (size_t)d * 6);
    size_t total = 2 * per_dir + 3 * R * d;
    total += (size_t)B * (Z + 2 * (size_t)Hh + m + 6 * (size_t)d);
    // chunk partials of all sixteen layer products side by side
    const size_t widest = 2 * (((size_t)d + F + 1) * Hf + ((size_t)Hf + 1) * d + ((size_t)d + 1) * Hg + ((size_t)Hg + 1) * d) +
                          3 * ((E + 1) * (size_t)d + ((size_t)d + 1) * d) + (Z + 1) * (size_t)Hh + ((size_t)Hh + 1) * m;
    return total + (size_t)kGradChunks * widest + 256;
}

cudaError_t launch_policy_gradient(GradArgs a, const DeviceInfo &di, float *ws, cudaStream_t stream) {
    const int n = a.n, B = a.B, d = a.d, F = a.F, m = a.m;
    const size_t R = (size_t)n * B;
    const int Z = 5 * d + F, Hh = a.head.hidden_dim;
    float *p = ws;
    auto take = [&](size_t floats) { float *q = p; p += (floats + 3) & ~size_t(3); return q; };
    for (int dir = 0; dir < 2; ++dir) {
        const int Hf = a.f[dir].hidden_dim, Hg = a.g[dir].hidden_dim;
        a.FH[dir] = take(R * Hf); a.DFH[dir] = take(R * Hf);
        a.T1[dir] = take(R * Hg); a.DT1[dir] = take(R * Hg);
        a.M[dir] = take(R * d); a.DS[dir] = take(R * d);
        a.DPRE_F2[dir] = take(R * d); a.DPRE_G2[dir] = take(R * d);
        a.Sg[dir] = take(R * d); a.DH[dir] = take(R * d);
    }
    for (int i = 0; i < 3; ++i) a.DPRE_L[i] = take(R * d);
    a.Zbuf = take((size_t)B * Z); a.HID = take((size_t)B * Hh); a.DHID = take((size_t)B * Hh);
    a.DLOG = take((size_t)B * m); a.Sbuf = take((size_t)B * 3 * d); a.DPRE_H = take((size_t)B * 3 * d);
    float *partial = p;

    cudaError_t err = cudaMemsetAsync(a.DPRE_L[0], 0, 3 * ((R * d + 3) & ~size_t(3)) * sizeof(float), stream);
    if (err != cudaSuccess) return err;
    // 1. messages
    {
        const int Hf = std::max(a.f[0].hidden_dim, a.f[1].hidden_dim);
        const size_t smem = (size_t)kRows * (d + F + Hf) * sizeof(float);
        err = cudaFuncSetAttribute(grad_messages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        const int blocks = (int)std::min<size_t>((R + kRows - 1) / kRows, 4 * (size_t)di.sm_count);
        grad_messages_kernel<<<dim3(blocks, 2), kThreads, smem, stream>>>(a);
        count_launch();
    }
    // 2. head and pooling
    {
        const size_t E = 2 * (size_t)d + F;
        const size_t floats = 2 * (size_t)Z + 2 * (size_t)Hh + 6 * (size_t)d + ((m + 3) & ~3) +
                              (size_t)(kThreads / 32) * 3 * d + (size_t)(kThreads / 32) * ((E + 3) & ~size_t(3)) +
                              3 * (E * d + d);
        const size_t smem = floats * sizeof(float);
        err = cudaFuncSetAttribute(grad_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        grad_head_kernel<<<std::min(B, 8 * di.sm_count), kThreads, smem, stream>>>(a);
        count_launch();
    }
    // 3. reverse sweeps
    {
        const int slices = std::max(1, std::min(B, di.sm_count / 2));
        const int S = (B + slices - 1) / slices;
        int W = d;
        for (int dir = 0; dir < 2; ++dir) W = std::max({W, a.f[dir].hidden_dim, a.g[dir].hidden_dim});
        size_t wfloats = 0;
        for (int dir = 0; dir < 2; ++dir) {
            const size_t Hf = a.f[dir].hidden_dim, Hg = a.g[dir].hidden_dim;
            const size_t pd = ((size_t)d + 3) & ~size_t(3), pf = (Hf + 3) & ~size_t(3), pg = (Hg + 3) & ~size_t(3);
            wfloats = std::max(wfloats, d * pf + Hf * pd + 2 * d * pg + Hg * pd + Hg);
        }
        W |= 1;
        const size_t smem = (7 * (size_t)kSweepRows * W + wfloats) * sizeof(float);
        if (smem > (size_t)di.max_smem_optin) return cudaErrorNotSupported;
        err = cudaFuncSetAttribute(grad_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        grad_sweep_kernel<<<dim3((B + S - 1) / S, 2), kThreads, smem, stream>>>(a, S);
        count_launch();
    }
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    // 4. weight gradients: dW = in^T dpre, db = sum dpre, every layer in one launch
    // two launches: the layers summed over all (node, state) rows, and those summed over
    // states only (the head's wide matrices would otherwise set every block's shared memory)
    WeightJobs by_row, by_state;
    by_row.count = by_state.count = 0;
    auto job = [&](const float *in0, int w0, int s0, const float *in1, int w1, const float *in2, int w2,
                   const float *dp, int dp_stride, int J, size_t rows, float *dW, float *db) {
        WeightJobs &list = rows == R ? by_row : by_state;
        WeightJob &w = list.job[list.count++];
        w.in[0] = in0; w.in[1] = in1; w.in[2] = in2;
        w.width[0] = w0; w.width[1] = w1; w.width[2] = w2;
        w.stride[0] = s0; w.stride[1] = w1; w.stride[2] = w2;
        w.dp = dp; w.dp_stride = dp_stride; w.K = w0 + w1 + w2; w.J = J; w.R = rows;
        w.dW = dW; w.db = db;
        w.accumulate = a.accumulate;
        w.chunks = (int)std::max<size_t>(1, std::min<size_t>(kGradChunks, (rows + kRows - 1) / kRows));
        w.partial = partial;                                  // each job its own stretch
        partial += (size_t)w.chunks * (w.K + 1) * w.J;
    };
    for (int dir = 0; dir < 2; ++dir) {
        const int Hf = a.f[dir].hidden_dim, Hg = a.g[dir].hidden_dim;
        job(a.H[dir], d, d, a.X, F, nullptr, 0, a.DFH[dir], Hf, Hf, R, a.gf[dir].W1, a.gf[dir].b1);
        job(a.FH[dir], Hf, Hf, nullptr, 0, nullptr, 0, a.DPRE_F2[dir], d, d, R, a.gf[dir].W2, a.gf[dir].b2);
        job(a.Sg[dir], d, d, nullptr, 0, nullptr, 0, a.DT1[dir], Hg, Hg, R, a.gg[dir].W1, a.gg[dir].b1);
        job(a.T1[dir], Hg, Hg, nullptr, 0, nullptr, 0, a.DPRE_G2[dir], d, d, R, a.gg[dir].W2, a.gg[dir].b2);
    }
    for (int i = 0; i < 3; ++i) {
        job(a.H[0], d, d, a.H[1], d, a.X, F, a.DPRE_L[i], d, d, R, a.gl[i].W1, a.gl[i].b1);
        // h_i: rows are states; the inputs and gradients of set i sit at column offset i * d of [B][3][d]
        job(a.Sbuf + i * d, d, 3 * d, nullptr, 0, nullptr, 0, a.DPRE_H + i * d, 3 * d, d, B, a.gh[i].W1, a.gh[i].b1);
    }
    job(a.Zbuf, Z, Z, nullptr, 0, nullptr, 0, a.DHID, Hh, Hh, B, a.ghead.W1, a.ghead.b1);
    job(a.HID, Hh, Hh, nullptr, 0, nullptr, 0, a.DLOG, m, m, B, a.ghead.W2, a.ghead.b2);
    err = weight_grads(by_row, stream);
    if (err != cudaSuccess) return err;
    return weight_grads(by_state, stream);
}

}  // namespace placeto
