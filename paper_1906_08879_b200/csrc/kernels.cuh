// Device-side argument structs and launcher declarations shared by the
// library's translation units.
#pragma once
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstdint>

#include "placeto.h"

namespace placeto {

// One direction's level schedule in device memory (see placeto_graph_host_view).
struct DevLevels {
    int n_levels;
    const int *level_ptr, *order, *nbr_ptr, *nbr;
    int n_slots;                     // on-chip message slots (see plan.h)
    const int *own_slot, *nbr_slot;
    int n_nbr;                       // total neighbour entries
    // packed records for kernels that stream the schedule level by level:
    //   lvl4[level] = {first position, width, first neighbour entry, neighbour entries of the level}
    //   pos4[p]     = {first neighbour entry, end of neighbour entries, own slot, node id}
    const int4 *lvl4, *pos4;
    int max_level_nbr;               // most neighbour entries in one level
};

// One feed-forward network with device pointers.
struct DevMlp {
    int n_layers, in_dim, hidden_dim, out_dim, act, final_act;
    const float *W1, *b1, *W2, *b2;
};

inline DevMlp to_dev(const placeto_mlp &m) {
    DevMlp d;
    d.n_layers = m.n_layers;
    d.in_dim = m.in_dim;
    d.hidden_dim = m.n_layers == 2 ? m.hidden_dim : m.out_dim;
    d.out_dim = m.out_dim;
    d.act = m.act;
    d.final_act = m.final_act;
    d.W1 = m.W1; d.b1 = m.b1; d.W2 = m.W2; d.b2 = m.b2;
    return d;
}

// Floats a network occupies when staged contiguously (W1, b1, W2, b2).
inline size_t mlp_floats(const DevMlp &m) {
    size_t s = (size_t)m.in_dim * m.hidden_dim + m.hidden_dim;
    if (m.n_layers == 2) s += (size_t)m.hidden_dim * m.out_dim + m.out_dim;
    return s;
}

// Where a kernel reports a bounded wait that ran out (or, in a PLACETO_DEBUG build, an index
// out of range): a 16-byte record {magic, magic, call number, status code}. A record counts
// only if it carries the number of the call that asks, so nothing ever has to be cleared and
// whatever an uninitialised workspace holds cannot be mistaken for a report.
constexpr int kStatusMagic0 = 0x504c4143, kStatusMagic1 = 0x544f5354;
struct StatusSlot {
    int4 *record;   // device memory, 16-byte aligned (null: nowhere to report)
    int call;
};
#ifdef __CUDACC__
__device__ __forceinline__ void report_status(const StatusSlot &s, int code) {
    if (s.record != nullptr) *s.record = make_int4(kStatusMagic0, kStatusMagic1, s.call, code);
}
// Index checks of a library built with -DPLACETO_DEBUG (the stand-in for a memory checker):
// a schedule record, slot, node or state index out of range is reported as
// PLACETO_ERR_INVALID_ARG through the call's status record; nothing traps. The kernels test the
// records where they stage them, before any access uses them. Without the flag no code is made.
#ifdef PLACETO_DEBUG
#define PLACETO_DEBUG_CHECK(status, cond) \
    do { if (!(cond)) placeto::report_status((status), PLACETO_ERR_INVALID_ARG); } while (0)
#else
#define PLACETO_DEBUG_CHECK(status, cond) do { } while (0)
#endif
#endif

// Compact placement states (Sec. 2.1): per (node, state) one byte - the node's device in
// the low six bits, bit 7 set once the node has been visited - and the current node per
// state. Together with the per-node cost and output size they determine every raw feature
// (Sec. 2.2 step 1), so a kernel given them builds x on the fly instead of reading X:
// one byte instead of 4 F per node and state.
struct CompactState {
    const float *cost, *bytes;   // [n]
    const uint8_t *state;        // [n][B]; null: the features come from X
    const int *cur;              // [B]
    int m;
};
#ifdef __CUDACC__
// feature k of node v in state b: [cost, bytes, one-hot_m(device), v == cur, visited]
__device__ __forceinline__ float compact_feature(const CompactState &c, int v, int b, int B, int k) {
    if (k == 0) return c.cost[v];
    if (k == 1) return c.bytes[v];
    const unsigned s = c.state[(size_t)v * B + b];
    if (k < 2 + c.m) return (int)(s & 63u) == k - 2 ? 1.f : 0.f;
    if (k == 2 + c.m) return c.cur[b] == v ? 1.f : 0.f;
    return (float)(s >> 7);
}
// all F = m + 4 features of node v in state b into x[0 .. F): one state byte, the node's cost and
// size, the state's current node
__device__ __forceinline__ void compact_features(const CompactState &c, int v, int b, int B, float *x) {
    const unsigned s = c.state[(size_t)v * B + b];
    const int dev = (int)(s & 63u);
    x[0] = c.cost[v];
    x[1] = c.bytes[v];
    for (int k = 0; k < c.m; ++k) x[2 + k] = k == dev ? 1.f : 0.f;
    x[2 + c.m] = c.cur[b] == v ? 1.f : 0.f;
    x[3 + c.m] = (float)(s >> 7);
}
#endif

// The MDP transition fused into the head kernel (episodes on compact states): after the
// logits of step t the thread of a state picks the device of the current node (argmax, or
// the inverse CDF of the FP32 softmax at uniforms[e][t]), records it, marks the node visited
// and makes order[t + 1] current.
struct EpisodeStep {
    int enabled, t, n;
    const int *order;          // [n]
    const float *uniforms;     // [E][n] or null (greedy)
    uint8_t *state;            // [n][E] compact states, updated in place
    int *cur;                  // [E], updated in place
    float *logp;               // [E][n] by step, or null
    uint8_t *actions;          // [E][n] by step, or null
};

struct EmbedArgs {
    DevLevels lv[2];
    DevMlp f[2], g[2];
    const float *X;
    float *H[2];   // outputs [n][B][d]
    float *M[2];   // messages f([h || x]) per node and state, [n][B][d] (workspace)
    int n, B, F, d;
    int max_level_width;   // widest level over both directions
    StatusSlot status;
    CompactState compact;  // compact.state != null: X is not read
};

struct PoolArgs {
    DevMlp l[3], h[3], head;
    const float *X, *H[2];
    const int *cur;
    const uint8_t *relation;   // [n][n]
    float *partial;            // [chunks][B][3][d] (workspace)
    float *logits, *probs;     // [B][m]; probs may be null
    int n, B, F, d, m;
    int chunks, chunk_nodes;
    StatusSlot status;
    CompactState compact;  // compact.state != null: X is not read
    EpisodeStep step;      // step.enabled: the head kernel also makes the MDP transition
};

struct EpisodeArgs {
    int n, E, m;
    const int *order;          // [n] node visited at step t
    const float *uniforms;     // [E][n] or null (greedy)
    const float *logits;       // [E][m] of the current step
    uint8_t *dev, *placed;     // [E][n]
    int *cur;                  // [E]
    float *logp;               // [E][n] by step, or null
    uint8_t *actions;          // [E][n] by step, or null
    float *X;                  // [n][E][m + 4] raw features, patched in place after every step
};

struct SimArgs {
    int n, n_edges, m, P;
    const int *child_ptr, *child, *n_parents;   // by node id
    const int *parent_ptr, *parent;             // by node id, ascending
    const float *cost, *bytes;                  // [n]
    const uint8_t *dev;                         // [P][n]
    double bandwidth;
    double mem_limit, mem_scale;                // M and c of the memory-penalised run time
    double *runtime;                            // [P] or null
    double *peak_memory;                        // [P][m] or null
    double *penalised;                          // [P] or null
    char *workspace;
};

// Policy gradient (gradient.cu): inputs, per-row intermediates in the workspace, outputs.
constexpr int kGradChunks = 256;   // row chunks whose partial weight gradients are added in order
struct GradOut { float *W1, *b1, *W2, *b2; };
struct GradArgs {
    int n, B, d, F, m;
    const uint8_t *relation;
    DevLevels lv[2];
    const int *child_ptr, *child, *parent_ptr, *parent;   // by node id
    DevMlp f[2], g[2], l[3], h[3], head;
    const float *X, *H[2];
    const int *cur, *actions;
    const float *advantages;
    float beta;
    int accumulate;            // 1: gradients are added to the output buffers
    float *FH[2], *DFH[2], *T1[2], *DT1[2], *M[2], *DS[2], *DPRE_F2[2], *DPRE_G2[2], *Sg[2], *DH[2];
    float *DPRE_L[3], *Zbuf, *HID, *DHID, *DLOG, *Sbuf, *DPRE_H;
    GradOut gf[2], gg[2], gl[3], gh[3], ghead;
};

struct DeviceInfo {
    int sm_count;
    int max_smem_optin;   // bytes per block
};

// Counts launches of the calling thread's current forward call.
void count_launch(int k = 1);

#ifdef __CUDACC__
// ---- bulk asynchronous copies (the TMA unit moves a contiguous run of bytes from
// global to shared memory and reports the bytes on an mbarrier) -------------------
__device__ __forceinline__ unsigned smem_addr(const void *p) {
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned long long *bar, int arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect(unsigned long long *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
// src and dst 16-byte aligned, bytes a positive multiple of 16
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned bytes,
                                          unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst)),
        "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}
// Waits for phase `parity` of the barrier; gives up after a bounded number of
// polls (a copy that never lands must not hang the device) and reports it.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity) {
    for (int i = 0; i < (1 << 22); ++i) {
        unsigned done;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}"
            : "=r"(done)
            : "r"(smem_addr(bar)), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

#endif

// Programmatic dependent launch. Inside one forward call the library's kernels
// follow each other on the stream; a kernel launched with launch_overlapped may
// start while its predecessor is still running and do the part of its set-up
// that reads nothing the predecessor writes (schedule staging, weights), then
// calls dependency_wait() before it touches the predecessor's output. The
// predecessor allows this with dependents_may_start(). Only launches whose
// predecessor is a kernel of this library use it: weights and other caller
// inputs may have been written by the caller's own previous kernel, which the
// first launch of every call waits for in the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dependents_may_start() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(bool overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// features.cu
cudaError_t launch_features(int n, int B, int m, const float *cost, const float *bytes,
                            const uint8_t *dev, const int *cur, const uint8_t *placed, float *X,
                            cudaStream_t stream, bool overlap = false);

// Copies five host-resident, device-addressable buffers into device memory in one launch.
cudaError_t launch_stage_inputs(const void *const (&src)[5], void *const (&dst)[5],
                                const size_t (&bytes)[5], int sm_count, cudaStream_t stream);

// episode.cu: the MDP transition between two policy evaluations of an episode
cudaError_t launch_episode_begin(const EpisodeArgs &a, cudaStream_t stream);
cudaError_t launch_episode_step(const EpisodeArgs &a, int t, cudaStream_t stream);
// compact states: state[v][e] from the initial placement dev[e][v] (nothing visited), cur[e] = order[0];
// and back: dev[e][v] = the device of state[v][e]
cudaError_t launch_episode_begin_compact(int n, int E, const int *order, const uint8_t *dev, uint8_t *state,
                                         int *cur, cudaStream_t stream);
cudaError_t launch_episode_end_compact(int n, int E, const uint8_t *state, uint8_t *dev, cudaStream_t stream);
// true when an episode step on these shapes runs on kernels that take compact states
bool pool_head_takes_compact(const PoolArgs &a);

// simulator.cu: event-based run time of P placements, one thread each
size_t sim_workspace_bytes(int n, int n_edges, int m, int P);
cudaError_t launch_simulator(const SimArgs &a, cudaStream_t stream);

// gradient.cu: gradient of the policy objective with respect to all weights
bool policy_gradient_applicable(const GradArgs &a);
size_t policy_gradient_workspace_floats(int n, int B, int d, int F, int m, int Hf, int Hg, int Hh);
cudaError_t launch_policy_gradient(GradArgs a, const DeviceInfo &di, float *ws, cudaStream_t stream);

// writes the d x d identity matrix followed by d zeros (an identity layer: W2 = I, b2 = 0)
cudaError_t launch_identity_layer(float *dst, int d, cudaStream_t stream);

// embed_generic.cu: dimension-generic message passing. schedule is one of
// PLACETO_PER_LEVEL / PLACETO_SLICED / PLACETO_COOPERATIVE.
cudaError_t launch_embed_generic(const EmbedArgs &a, const DeviceInfo &di, unsigned schedule,
                                 cudaStream_t stream);

// the synchronous k-round form of step 2 on the generic kernel (rounds + 1 launches);
// msg: four [n][B][d] buffers, two per direction
cudaError_t launch_embed_rounds(const EmbedArgs &a, const DeviceInfo &di, int rounds, float *const msg[4],
                                cudaStream_t stream);

// embed_rounds_d32.cu: the same rounds for the shapes of embed_d32_applicable (throughput kernel)
cudaError_t launch_embed_rounds_d32(const EmbedArgs &a, const DeviceInfo &di, int rounds,
                                    float *const msg[4], cudaStream_t stream);

// embed_d32.cu: specialised message passing for d = 32 with two-layer ReLU
// networks of hidden width 32; returns cudaErrorNotSupported when the shapes or
// the shared-memory budget do not fit (the caller then uses the generic kernel).
bool embed_d32_applicable(const EmbedArgs &a);
bool embed_d32_fits(const EmbedArgs &a, const DeviceInfo &di);   // applicable and within shared memory
cudaError_t launch_embed_d32(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream,
                             bool overlap = false);

// embed_d64.cu: the same for d = 64 (four-warp column-split groups, both
// directions in one block).
bool embed_d64_applicable(const EmbedArgs &a);
cudaError_t launch_embed_d64(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream);

// embed_mma.cu: d = 32 / 64 on the tensor cores (mma.sync, TF32 operands split
// into head + tail, three products per step for FP32 accuracy).
bool embed_mma_applicable(const EmbedArgs &a);
bool embed_mma_preferred(const EmbedArgs &a);   // applicable and faster than the FMA kernels
cudaError_t launch_embed_mma(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream,
                             bool overlap = false);

// embed_pipe.cu: d = 64 as a pipeline of layers on mma.sync (a group of warps per layer of f and g,
// tiles of eight rows handed from layer to layer through shared memory). cudaErrorNotSupported when
// the schedule and the message slots do not fit in shared memory.
bool embed_pipe_applicable(const EmbedArgs &a);
bool embed_pipe_preferred(const EmbedArgs &a, const DeviceInfo &di);   // where the library picks it
cudaError_t launch_embed_pipe(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap = false);

// embed_tc.cu: d = 64 on tcgen05 tensor cores with accumulators in tensor memory (TF32 head + tail
// operands, all four partial products per instruction). A bounded wait that runs out inside the
// kernel is reported through a.status as PLACETO_ERR_TIMEOUT.
bool embed_tc_applicable(const EmbedArgs &a);
cudaError_t launch_embed_tc(const EmbedArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap = false);

// A kernel whose only job is to let a bounded wait run out (a copy that delivers fewer bytes
// than the barrier expects, a poll limit of a few thousand tries) and report it: exercises the
// time-out path without faulting or hanging anything.
cudaError_t launch_wait_timeout_probe(const StatusSlot &status, cudaStream_t stream);

// aggregator.cu: the "simple aggregator" policy (no message passing, no sets), one block per state
cudaError_t launch_simple_aggregator(const DevMlp &l, const DevMlp &h, const DevMlp &head, const float *X, int n,
                                     int B, int F, int d, int m, float *logits, float *probs, const DeviceInfo &di,
                                     cudaStream_t stream);

// policy_generic.cu: pooling partial sums, then per-state finalisation + head + softmax.
int pool_chunks(int n, int B, const DeviceInfo &di);
cudaError_t launch_policy_generic(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream);
// adds the chunk partial sums, applies h_i, the head and the softmax (one block per state)
cudaError_t launch_pool_head(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream);

// policy_d32.cu: specialised partial sums for d = 32, F a multiple of 4, single-layer ReLU l_i
bool pool_d32_applicable(const PoolArgs &a);
bool pool_d32_fits(const PoolArgs &a, const DeviceInfo &di);      // applicable (a.chunk_nodes set) and within shared memory
void pool_d32_chunks(int n, int B, int F, const DeviceInfo &di, int *chunk_nodes, int *chunks);
cudaError_t launch_pool_d32(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream,
                            bool overlap = false);

// policy_d64.cu: the same for d = 64 (weights of all three sets split over the block's warps)
bool pool_d64_applicable(const PoolArgs &a);
void pool_d64_chunks(int n, int B, int F, const DeviceInfo &di, int *chunk_nodes, int *chunks);
cudaError_t launch_pool_d64(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream,
                            bool overlap = false);

// policy_tc.cu: the same partial sums for d = 64 on tcgen05 tensor cores (weights of the current
// set in tensor memory, two operand tiles in shared memory, accumulators in tensor memory)
bool pool_tc_applicable(const PoolArgs &a);
void pool_tc_chunks(int n, int B, const DeviceInfo &di, int *chunk_nodes, int *chunks);
cudaError_t launch_pool_tc(const PoolArgs &a, const DeviceInfo &di, cudaStream_t stream, bool overlap = false);

}  // namespace placeto
