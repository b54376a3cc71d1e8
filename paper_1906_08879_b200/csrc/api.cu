// C ABI of the library (see include/placeto.h): argument validation, workspace
// layout, schedule selection and kernel launches. No arithmetic of the policy
// happens on the host.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "kernels.cuh"
#include "plan.h"

using namespace placeto;

struct placeto_graph {
    HostPlan host;
    bool on_device = false;
    int device = -1;
    DeviceInfo info{};
    int *d_ints = nullptr;       // one allocation for all int arrays
    int4 *d_packed = nullptr;    // per direction lvl4[n_levels], pos4[n] (see DevLevels)
    int *d_child_ptr = nullptr, *d_child = nullptr, *d_n_parents = nullptr;   // inside d_ints
    int *d_parent_ptr = nullptr, *d_parent = nullptr;                          // inside d_ints
    uint8_t *d_relation = nullptr;
    DevLevels lv[2]{};
    mutable std::atomic<int> calls{0};   // number of the latest forward call (see StatusSlot)
};

namespace placeto {

static thread_local int t_launches = 0;
void count_launch(int k) { t_launches += k; }

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;   // reserved at offset 0 of every workspace; the first 4 bytes are the status word
inline size_t align_up(size_t v) { return (v + kAlign - 1) & ~(kAlign - 1); }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool mlp_ok(const placeto_mlp &m, int in, int out) {
    if (m.n_layers != 1 && m.n_layers != 2) return false;
    if (m.in_dim != in || m.out_dim != out) return false;
    if (m.act != 0 && m.act != 1) return false;
    if (m.final_act != 0 && m.final_act != 1) return false;
    if (!m.W1 || !m.b1 || !aligned16(m.W1) || !aligned16(m.b1)) return false;
    if (m.n_layers == 2) {
        if (m.hidden_dim < 1 || m.hidden_dim > PLACETO_MAX_HIDDEN) return false;
        if (!m.W2 || !m.b2 || !aligned16(m.W2) || !aligned16(m.b2)) return false;
    }
    return true;
}

placeto_status dims_ok(const placeto_weights *w) {
    if (!w) return PLACETO_ERR_INVALID_ARG;
    if (w->d < 1 || w->F < 1 || w->m < 1) return PLACETO_ERR_INVALID_ARG;
    if (w->d > PLACETO_MAX_D || w->F > PLACETO_MAX_F || w->m > PLACETO_MAX_M + 4) // head width
        return PLACETO_ERR_UNSUPPORTED;
    return PLACETO_OK;
}

placeto_status embed_weights_ok(const placeto_weights *w) {
    placeto_status s = dims_ok(w);
    if (s != PLACETO_OK) return s;
    const int d = w->d, F = w->F;
    if (!mlp_ok(w->f_down, d + F, d) || !mlp_ok(w->f_up, d + F, d) || !mlp_ok(w->g_down, d, d) ||
        !mlp_ok(w->g_up, d, d))
        return PLACETO_ERR_INVALID_ARG;
    return PLACETO_OK;
}

placeto_status pool_weights_ok(const placeto_weights *w) {
    placeto_status s = dims_ok(w);
    if (s != PLACETO_OK) return s;
    const int d = w->d, F = w->F;
    for (int i = 0; i < 3; ++i)
        if (!mlp_ok(w->l[i], 2 * d + F, d) || !mlp_ok(w->h[i], d, d)) return PLACETO_ERR_INVALID_ARG;
    if (!mlp_ok(w->head, 5 * d + F, w->m)) return PLACETO_ERR_INVALID_ARG;
    return PLACETO_OK;
}

struct Layout {
    size_t status;                 // 256 bytes at the start: the status word of the call
    size_t msg[2], msg_alt[2], partial, X, H[2], cost, bytes, dev, placed, cur, logits, probs, total;
    size_t grad, grad_extra;       // gradient call: its intermediates; identity layers of single-layer f, g
    size_t compact;                // episode call: the compact states [n][E]
    int chunks, chunk_nodes;       // node chunks of the generic pooling kernel
    int chunks32, chunk_nodes32;   // and of the d = 32 / d = 64 kernel (0 when neither can apply)
    int chunks_tc, chunk_nodes_tc; // and of the d = 64 tensor-core kernel (0 when it cannot apply)
};

// Workspace layout shared by every call; a call uses the leading part it needs.
Layout make_layout(const placeto_graph *g, const placeto_weights *w, int B, placeto_call call) {
    Layout L{};
    const size_t n = (size_t)g->host.n, d = (size_t)w->d, F = (size_t)w->F, m = (size_t)w->m;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.status = take(kStatusBytes);
    int chunks = pool_chunks((int)n, B, g->info);
    L.chunk_nodes = ((int)n + chunks - 1) / chunks;
    L.chunks = ((int)n + L.chunk_nodes - 1) / L.chunk_nodes;
    if (call == PLACETO_CALL_EMBED || call == PLACETO_CALL_EMBED_ROUNDS ||
        (call >= PLACETO_CALL_FORWARD && call <= PLACETO_CALL_EPISODE)) {
        L.msg[0] = take(n * B * d * sizeof(float));
        L.msg[1] = take(n * B * d * sizeof(float));
    }
    if (call == PLACETO_CALL_GRADIENT) {
        // a single-layer network is differentiated as the two-layer network it equals (see
        // placeto_policy_gradient): its hidden width is then its output width
        auto hidden = [](const placeto_mlp &net) { return net.n_layers == 2 ? net.hidden_dim : net.out_dim; };
        const int Hf = std::max(hidden(w->f_down), hidden(w->f_up));
        const int Hg = std::max(hidden(w->g_down), hidden(w->g_up));
        L.grad = take(policy_gradient_workspace_floats((int)n, B, w->d, w->F, w->m, Hf, Hg, w->head.hidden_dim) *
                      sizeof(float));
        L.grad_extra = take(4 * 2 * (d * d + d) * sizeof(float));
        L.total = off;
        return L;
    }
    if (call == PLACETO_CALL_EMBED_ROUNDS) {
        L.msg_alt[0] = take(n * B * d * sizeof(float));
        L.msg_alt[1] = take(n * B * d * sizeof(float));
        L.total = off;
        return L;
    }
    if (w->F >= 4 && w->F <= 16 && (w->F & 3) == 0) {
        if (w->d == 32) pool_d32_chunks((int)n, B, w->F, g->info, &L.chunk_nodes32, &L.chunks32);
        if (w->d == 64) pool_d64_chunks((int)n, B, w->F, g->info, &L.chunk_nodes32, &L.chunks32);
        if (w->d == 64) pool_tc_chunks((int)n, B, g->info, &L.chunk_nodes_tc, &L.chunks_tc);
    }
    if (call == PLACETO_CALL_LOGITS || (call >= PLACETO_CALL_FORWARD && call <= PLACETO_CALL_EPISODE))
        L.partial = take((size_t)std::max(L.chunks, std::max(L.chunks32, L.chunks_tc)) * B * 3 * d * sizeof(float));
    if (call >= PLACETO_CALL_FORWARD && call <= PLACETO_CALL_EPISODE) {
        L.X = take(n * B * F * sizeof(float));
        L.H[0] = take(n * B * d * sizeof(float));
        L.H[1] = take(n * B * d * sizeof(float));
    }
    if (call == PLACETO_CALL_FORWARD_HOST) {
        L.cost = take(n * sizeof(float));
        L.bytes = take(n * sizeof(float));
        L.dev = take(n * B);
        L.placed = take(n * B);
        L.cur = take((size_t)B * sizeof(int32_t));
        L.logits = take((size_t)B * m * sizeof(float));
        L.probs = take((size_t)B * m * sizeof(float));
    }
    if (call == PLACETO_CALL_EPISODE) {
        L.compact = take(n * B);
        L.placed = take(n * B);
        L.cur = take((size_t)B * sizeof(int32_t));
        L.logits = take((size_t)B * m * sizeof(float));
        L.probs = take((size_t)B * m * sizeof(float));
    }
    L.total = off;
    return L;
}

unsigned pick_schedule(unsigned flags) {
    if (flags & PLACETO_PER_LEVEL) return PLACETO_PER_LEVEL;
    if (flags & PLACETO_COOPERATIVE) return PLACETO_COOPERATIVE;
    return PLACETO_SLICED;
}

bool flags_ok(uint32_t flags) {
    const uint32_t known = PLACETO_PER_LEVEL | PLACETO_SLICED | PLACETO_COOPERATIVE |
                           PLACETO_GENERIC | PLACETO_FMA_ONLY | PLACETO_TENSOR | PLACETO_TCGEN05 | PLACETO_PIPELINE;
    if (flags & ~known) return false;
    const uint32_t sched = flags & (PLACETO_PER_LEVEL | PLACETO_SLICED | PLACETO_COOPERATIVE);
    return (sched & (sched - 1)) == 0;   // at most one schedule
}

// The device-side address of a page-locked (cudaHostAlloc / cudaHostRegister) host
// buffer, or nullptr when the pointer is pageable host memory or anything else.
const void *device_alias(const void *p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// The report slot of a new call on `g`: the record at the start of the workspace (or of the
// built-in scratch) tagged with the call's number.
StatusSlot new_status_slot(const placeto_graph *g, char *ws, const Layout &L) {
    StatusSlot s;
    s.record = reinterpret_cast<int4 *>(ws + L.status);
    s.call = g->calls.fetch_add(1) + 1;
    return s;
}

placeto_status cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return PLACETO_OK;
    if (e == cudaErrorCooperativeLaunchTooLarge) return PLACETO_ERR_UNSUPPORTED;
    return PLACETO_ERR_CUDA;
}

placeto_status run_embed(const placeto_graph *g, const placeto_weights *w, const float *X, int B,
                         float *H_down, float *H_up, char *ws, const Layout &L, uint32_t flags,
                         cudaStream_t stream, const StatusSlot &status, bool after_own_kernel = false,
                         const CompactState *compact = nullptr) {
    EmbedArgs a;
    a.status = status;
    a.compact = compact ? *compact : CompactState{};
    a.lv[0] = g->lv[0]; a.lv[1] = g->lv[1];
    a.f[0] = to_dev(w->f_down); a.f[1] = to_dev(w->f_up);
    a.g[0] = to_dev(w->g_down); a.g[1] = to_dev(w->g_up);
    a.X = X;
    a.H[0] = H_down; a.H[1] = H_up;
    a.M[0] = reinterpret_cast<float *>(ws + L.msg[0]);
    a.M[1] = reinterpret_cast<float *>(ws + L.msg[1]);
    a.n = g->host.n; a.B = B; a.F = w->F; a.d = w->d;
    a.max_level_width = g->host.max_level_width;
    const unsigned schedule = pick_schedule(flags);
    if (compact != nullptr)      // only the d = 32 kernel builds features from compact states
        return cuda_status(launch_embed_d32(a, g->info, stream, after_own_kernel));
    if ((flags & PLACETO_TCGEN05) && !(flags & (PLACETO_GENERIC | PLACETO_FMA_ONLY)) &&
        schedule == PLACETO_SLICED && embed_tc_applicable(a)) {
        cudaError_t e = launch_embed_tc(a, g->info, stream, after_own_kernel);
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    // d = 64: the pipeline of layers, if it fits
    if (!(flags & (PLACETO_GENERIC | PLACETO_FMA_ONLY | PLACETO_TENSOR)) && schedule == PLACETO_SLICED &&
        ((flags & PLACETO_PIPELINE) ? embed_pipe_applicable(a) : embed_pipe_preferred(a, g->info))) {
        cudaError_t e = launch_embed_pipe(a, g->info, stream, after_own_kernel);
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    const bool want_mma = (flags & PLACETO_TENSOR) ? embed_mma_applicable(a) : embed_mma_preferred(a);
    if (!(flags & (PLACETO_GENERIC | PLACETO_FMA_ONLY)) && schedule == PLACETO_SLICED && want_mma) {
        cudaError_t e = launch_embed_mma(a, g->info, stream, after_own_kernel);
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    if (!(flags & PLACETO_GENERIC) && schedule == PLACETO_SLICED && embed_d32_applicable(a)) {
        cudaError_t e = launch_embed_d32(a, g->info, stream, after_own_kernel);
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    if (!(flags & PLACETO_GENERIC) && schedule == PLACETO_SLICED && embed_d64_applicable(a)) {
        cudaError_t e = launch_embed_d64(a, g->info, stream);
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    return cuda_status(launch_embed_generic(a, g->info, schedule, stream));
}

placeto_status run_pool(const placeto_graph *g, const placeto_weights *w, const float *X,
                        const float *H_down, const float *H_up, const int32_t *cur, int B,
                        float *logits, float *probs, char *ws, const Layout &L, uint32_t flags,
                        cudaStream_t stream, const StatusSlot &status, bool after_own_kernel = false,
                        const CompactState *compact = nullptr, const EpisodeStep *step = nullptr) {
    PoolArgs a;
    a.status = status;
    a.compact = compact ? *compact : CompactState{};
    a.step = step ? *step : EpisodeStep{};
    for (int i = 0; i < 3; ++i) { a.l[i] = to_dev(w->l[i]); a.h[i] = to_dev(w->h[i]); }
    a.head = to_dev(w->head);
    a.X = X; a.H[0] = H_down; a.H[1] = H_up;
    a.cur = cur;
    a.relation = g->d_relation;
    a.partial = reinterpret_cast<float *>(ws + L.partial);
    a.logits = logits; a.probs = probs;
    a.n = g->host.n; a.B = B; a.F = w->F; a.d = w->d; a.m = w->m;
    const bool fast32 = pool_d32_applicable(a), fast64 = pool_d64_applicable(a);
    if (compact != nullptr) {    // only the d = 32 kernel and the fast head kernel take compact states
        a.chunks = L.chunks32; a.chunk_nodes = L.chunk_nodes32;
        cudaError_t e = launch_pool_d32(a, g->info, stream, after_own_kernel);
        return cuda_status(e == cudaSuccess ? launch_pool_head(a, g->info, stream) : e);
    }
    if (!(flags & (PLACETO_GENERIC | PLACETO_FMA_ONLY)) && L.chunks_tc > 0 && pool_tc_applicable(a)) {
        a.chunks = L.chunks_tc; a.chunk_nodes = L.chunk_nodes_tc;
        cudaError_t e = launch_pool_tc(a, g->info, stream, after_own_kernel);
        if (e == cudaSuccess) return cuda_status(launch_pool_head(a, g->info, stream));
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    if (!(flags & PLACETO_GENERIC) && L.chunks32 > 0 && (fast32 || fast64)) {
        a.chunks = L.chunks32; a.chunk_nodes = L.chunk_nodes32;
        cudaError_t e = fast32 ? launch_pool_d32(a, g->info, stream, after_own_kernel)
                               : launch_pool_d64(a, g->info, stream, after_own_kernel);
        if (e == cudaSuccess) return cuda_status(launch_pool_head(a, g->info, stream));
        if (e != cudaErrorNotSupported) return cuda_status(e);
    }
    a.chunks = L.chunks; a.chunk_nodes = L.chunk_nodes;
    return cuda_status(launch_policy_generic(a, g->info, stream));
}

// The graph's arrays, the caller's buffers and the launch all belong to one device: the one
// that was current at placeto_graph_create must be current again.
bool on_graph_device(const placeto_graph *g) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == g->device;
}

placeto_status common_checks(const placeto_graph *g, int32_t B, const void *ws, size_t ws_bytes,
                             size_t need, uint32_t flags) {
    if (!g || !g->on_device || B < 1 || !flags_ok(flags)) return PLACETO_ERR_INVALID_ARG;
    if (!on_graph_device(g)) return PLACETO_ERR_INVALID_ARG;
    if ((size_t)B * g->host.n > (size_t)1 << 31) return PLACETO_ERR_UNSUPPORTED;
    if (!ws || !aligned16(ws)) return PLACETO_ERR_INVALID_ARG;
    if (ws_bytes < need) return PLACETO_ERR_WORKSPACE;
    return PLACETO_OK;
}

}  // namespace

// Scratch of placeto_policy_logits_static: part of the library image, one copy
// per device that loads it. In host code the symbol below is only a handle: the
// address a kernel can use comes from cudaGetSymbolAddress, looked up once per
// device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[PLACETO_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
char *g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on `device`, or nullptr on failure.
char *static_scratch_address(int device) {
    if (device < 0 || device >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_ptr[device]) return g_scratch_ptr[device];
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return nullptr;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return nullptr;
    void *ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess || !ptr) return nullptr;
    g_scratch_ptr[device] = static_cast<char *>(ptr);
    return g_scratch_ptr[device];
}

}  // namespace
}  // namespace placeto

extern "C" {

const char *placeto_status_string(placeto_status s) {
    switch (s) {
        case PLACETO_OK: return "ok";
        case PLACETO_ERR_INVALID_ARG: return "invalid argument";
        case PLACETO_ERR_NOT_DAG: return "edge list is not a DAG over [0, n)";
        case PLACETO_ERR_WORKSPACE: return "workspace too small";
        case PLACETO_ERR_UNSUPPORTED: return "unsupported dimensions or flag";
        case PLACETO_ERR_CUDA: return "CUDA error";
        case PLACETO_ERR_NO_MEMORY: return "out of memory";
        case PLACETO_ERR_SCRATCH_LIMIT: return "batch exceeds the built-in scratch of the no-allocation call";
        case PLACETO_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    }
    return "unknown status";
}

placeto_status placeto_graph_create(int32_t n, int64_t n_edges, const int32_t *src,
                                    const int32_t *dst, uint32_t flags, placeto_graph **out) {
    if (!out) return PLACETO_ERR_INVALID_ARG;
    *out = nullptr;
    if (flags & ~PLACETO_GRAPH_HOST_ONLY) return PLACETO_ERR_INVALID_ARG;
    placeto_graph *g = new (std::nothrow) placeto_graph();
    if (!g) return PLACETO_ERR_NO_MEMORY;
    placeto_status s = build_plan(n, n_edges, src, dst, g->host);
    if (s != PLACETO_OK) { delete g; return s; }
    if (flags & PLACETO_GRAPH_HOST_ONLY) { *out = g; return PLACETO_OK; }

    auto fail = [&](placeto_status st) {
        if (g->d_ints) cudaFree(g->d_ints);
        if (g->d_packed) cudaFree(g->d_packed);
        if (g->d_relation) cudaFree(g->d_relation);
        delete g;
        return st;
    };
    if (cudaGetDevice(&g->device) != cudaSuccess) return fail(PLACETO_ERR_CUDA);
    if (cudaDeviceGetAttribute(&g->info.sm_count, cudaDevAttrMultiProcessorCount, g->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&g->info.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, g->device) != cudaSuccess)
        return fail(PLACETO_ERR_CUDA);
    // one int allocation: per direction level_ptr, order, nbr_ptr, nbr, own_slot, nbr_slot
    // (each padded to 4 ints)
    constexpr int kArrays = 6;
    size_t total = 0;
    size_t offs[2][kArrays];
    for (int dir = 0; dir < 2; ++dir) {
        const LevelPlan &p = g->host.dir[dir];
        const size_t sizes[kArrays] = {p.level_ptr.size(), p.order.size(), p.nbr_ptr.size(),
                                       p.nbr.size(), p.own_slot.size(), p.nbr_slot.size()};
        for (int k = 0; k < kArrays; ++k) { offs[dir][k] = total; total += (sizes[k] + 3) & ~size_t(3); }
    }
    // and, by node id: children, parent counts (runtime simulator), parents (policy gradient)
    const std::vector<int32_t> *extra[5] = {&g->host.child_ptr, &g->host.child, &g->host.n_parents,
                                            &g->host.parent_ptr, &g->host.parent};
    size_t sim_off[5];
    for (int k = 0; k < 5; ++k) { sim_off[k] = total; total += (extra[k]->size() + 3) & ~size_t(3); }
    if (cudaMalloc(&g->d_ints, std::max<size_t>(total, 4) * sizeof(int)) != cudaSuccess)
        return fail(PLACETO_ERR_NO_MEMORY);
    if (cudaMalloc(&g->d_relation, g->host.relation.size()) != cudaSuccess)
        return fail(PLACETO_ERR_NO_MEMORY);
    for (int dir = 0; dir < 2; ++dir) {
        const LevelPlan &p = g->host.dir[dir];
        const std::vector<int32_t> *vecs[kArrays] = {&p.level_ptr, &p.order, &p.nbr_ptr,
                                                     &p.nbr, &p.own_slot, &p.nbr_slot};
        for (int k = 0; k < kArrays; ++k)
            if (!vecs[k]->empty() &&
                cudaMemcpy(g->d_ints + offs[dir][k], vecs[k]->data(), vecs[k]->size() * sizeof(int),
                           cudaMemcpyHostToDevice) != cudaSuccess)
                return fail(PLACETO_ERR_CUDA);
        g->lv[dir].n_levels = p.n_levels;
        g->lv[dir].level_ptr = g->d_ints + offs[dir][0];
        g->lv[dir].order = g->d_ints + offs[dir][1];
        g->lv[dir].nbr_ptr = g->d_ints + offs[dir][2];
        g->lv[dir].nbr = g->d_ints + offs[dir][3];
        g->lv[dir].n_slots = p.n_slots;
        g->lv[dir].own_slot = g->d_ints + offs[dir][4];
        g->lv[dir].nbr_slot = g->d_ints + offs[dir][5];
        g->lv[dir].n_nbr = static_cast<int>(p.nbr.size());
    }
    {
        int **dst[5] = {&g->d_child_ptr, &g->d_child, &g->d_n_parents, &g->d_parent_ptr, &g->d_parent};
        for (int k = 0; k < 5; ++k) {
            *dst[k] = g->d_ints + sim_off[k];
            if (!extra[k]->empty() &&
                cudaMemcpy(*dst[k], extra[k]->data(), extra[k]->size() * sizeof(int),
                           cudaMemcpyHostToDevice) != cudaSuccess)
                return fail(PLACETO_ERR_CUDA);
        }
    }
    if (cudaMemcpy(g->d_relation, g->host.relation.data(), g->host.relation.size(),
                   cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(PLACETO_ERR_CUDA);
    {   // packed per-level and per-position records (kernels that stream the schedule)
        std::vector<int4> packed;
        size_t at[2][2];
        for (int dir = 0; dir < 2; ++dir) {
            const LevelPlan &p = g->host.dir[dir];
            at[dir][0] = packed.size();
            int max_nbr = 0;
            for (int l = 0; l < p.n_levels; ++l) {
                const int p0 = p.level_ptr[l], p1 = p.level_ptr[l + 1];
                const int e0 = p.nbr_ptr[p0], e1 = p.nbr_ptr[p1];
                packed.push_back(make_int4(p0, p1 - p0, e0, e1 - e0));
                max_nbr = std::max(max_nbr, e1 - e0);
            }
            at[dir][1] = packed.size();
            for (int q = 0; q < g->host.n; ++q)
                packed.push_back(make_int4(p.nbr_ptr[q], p.nbr_ptr[q + 1], p.own_slot[q], p.order[q]));
            g->lv[dir].max_level_nbr = max_nbr;
        }
        if (cudaMalloc(&g->d_packed, packed.size() * sizeof(int4)) != cudaSuccess) return fail(PLACETO_ERR_NO_MEMORY);
        if (cudaMemcpy(g->d_packed, packed.data(), packed.size() * sizeof(int4), cudaMemcpyHostToDevice) != cudaSuccess)
            return fail(PLACETO_ERR_CUDA);
        for (int dir = 0; dir < 2; ++dir) {
            g->lv[dir].lvl4 = g->d_packed + at[dir][0];
            g->lv[dir].pos4 = g->d_packed + at[dir][1];
        }
    }
    g->on_device = true;
    *out = g;
    return PLACETO_OK;
}

placeto_status placeto_graph_info(const placeto_graph *g, int32_t *n, int64_t *n_edges,
                                  int32_t *n_levels_down, int32_t *n_levels_up,
                                  int32_t *max_level_width) {
    if (!g) return PLACETO_ERR_INVALID_ARG;
    if (n) *n = g->host.n;
    if (n_edges) *n_edges = g->host.n_edges;
    if (n_levels_down) *n_levels_down = g->host.dir[0].n_levels;
    if (n_levels_up) *n_levels_up = g->host.dir[1].n_levels;
    if (max_level_width) *max_level_width = g->host.max_level_width;
    return PLACETO_OK;
}

placeto_status placeto_graph_host_view(const placeto_graph *g, placeto_level_view *down,
                                       placeto_level_view *up, const uint8_t **relation) {
    if (!g) return PLACETO_ERR_INVALID_ARG;
    placeto_level_view *views[2] = {down, up};
    for (int dir = 0; dir < 2; ++dir) {
        if (!views[dir]) continue;
        const LevelPlan &p = g->host.dir[dir];
        views[dir]->n_levels = p.n_levels;
        views[dir]->level_ptr = p.level_ptr.data();
        views[dir]->order = p.order.data();
        views[dir]->nbr_ptr = p.nbr_ptr.data();
        views[dir]->nbr = p.nbr.data();
        views[dir]->n_slots = p.n_slots;
        views[dir]->own_slot = p.own_slot.data();
        views[dir]->nbr_slot = p.nbr_slot.data();
    }
    if (relation) *relation = g->host.relation.data();
    return PLACETO_OK;
}

void placeto_graph_destroy(placeto_graph *g) {
    if (!g) return;
    if (g->on_device) {
        int prev = -1;
        cudaGetDevice(&prev);
        if (prev != g->device) cudaSetDevice(g->device);
        cudaFree(g->d_ints);
        cudaFree(g->d_packed);
        cudaFree(g->d_relation);
        if (prev != g->device && prev >= 0) cudaSetDevice(prev);
    }
    delete g;
}

size_t placeto_workspace_bytes(const placeto_graph *g, const placeto_weights *w, int32_t B,
                               placeto_call call, uint32_t flags) {
    if (!g || !w || B < 1 || !flags_ok(flags) || dims_ok(w) != PLACETO_OK) return 0;
    if (call < PLACETO_CALL_EMBED || call > PLACETO_CALL_GRADIENT) return 0;
    if (call == PLACETO_CALL_GRADIENT && (embed_weights_ok(w) != PLACETO_OK || pool_weights_ok(w) != PLACETO_OK))
        return 0;
    placeto_graph tmp_info;   // HOST_ONLY graphs have no device info: assume a full B200
    const placeto_graph *use = g;
    if (!g->on_device) {
        tmp_info.host.n = g->host.n;
        tmp_info.info.sm_count = 148;
        tmp_info.info.max_smem_optin = 227 * 1024;
        use = &tmp_info;
    }
    return std::max<size_t>(make_layout(use, w, B, call).total, kAlign);
}

placeto_status placeto_build_features(const placeto_graph *g, const float *cost,
                                      const float *bytes, const uint8_t *dev, const int32_t *cur,
                                      const uint8_t *placed, int32_t m, int32_t B, float *X,
                                      void *stream) {
    t_launches = 0;
    if (!g || !g->on_device || B < 1 || m < 1 || m > PLACETO_MAX_M) return PLACETO_ERR_INVALID_ARG;
    if (!on_graph_device(g)) return PLACETO_ERR_INVALID_ARG;
    g->calls.fetch_add(1);
    if (!cost || !bytes || !dev || !cur || !placed || !X) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(bytes) || !aligned16(dev) || !aligned16(cur) ||
        !aligned16(placed) || !aligned16(X))
        return PLACETO_ERR_INVALID_ARG;
    return cuda_status(launch_features(g->host.n, B, m, cost, bytes, dev, cur, placed, X,
                                       static_cast<cudaStream_t>(stream)));
}

placeto_status placeto_embed_forward(const placeto_graph *g, const placeto_weights *w,
                                     const float *X, int32_t B, float *H_down, float *H_up,
                                     void *workspace, size_t workspace_bytes, uint32_t flags,
                                     void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1) return PLACETO_ERR_INVALID_ARG;
    const Layout L = make_layout(g, w, B, PLACETO_CALL_EMBED);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, flags);
    if (s != PLACETO_OK) return s;
    if (!X || !H_down || !H_up || !aligned16(X) || !aligned16(H_down) || !aligned16(H_up))
        return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    return run_embed(g, w, X, B, H_down, H_up, ws, L, flags, static_cast<cudaStream_t>(stream),
                     new_status_slot(g, ws, L));
}

placeto_status placeto_policy_logits(const placeto_graph *g, const placeto_weights *w,
                                     const float *X, const float *H_down, const float *H_up,
                                     const int32_t *cur, int32_t B, float *logits, float *probs,
                                     void *workspace, size_t workspace_bytes, uint32_t flags,
                                     void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1) return PLACETO_ERR_INVALID_ARG;
    const Layout L = make_layout(g, w, B, PLACETO_CALL_LOGITS);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, flags);
    if (s != PLACETO_OK) return s;
    if (!X || !H_down || !H_up || !cur || !logits) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(H_down) || !aligned16(H_up) || !aligned16(cur) ||
        !aligned16(logits) || (probs && !aligned16(probs)))
        return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    return run_pool(g, w, X, H_down, H_up, cur, B, logits, probs, ws, L, flags,
                    static_cast<cudaStream_t>(stream), new_status_slot(g, ws, L));
}

placeto_status placeto_policy_forward(const placeto_graph *g, const placeto_weights *w,
                                      const float *cost, const float *bytes, const uint8_t *dev,
                                      const int32_t *cur, const uint8_t *placed, int32_t B,
                                      float *logits, float *probs, void *workspace,
                                      size_t workspace_bytes, uint32_t flags, void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s == PLACETO_OK) s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1 || w->m > PLACETO_MAX_M || w->F != w->m + 4) return PLACETO_ERR_INVALID_ARG;
    const Layout L = make_layout(g, w, B, PLACETO_CALL_FORWARD);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, flags);
    if (s != PLACETO_OK) return s;
    if (!cost || !bytes || !dev || !cur || !placed || !logits) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(bytes) || !aligned16(dev) || !aligned16(cur) ||
        !aligned16(placed) || !aligned16(logits) || (probs && !aligned16(probs)))
        return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *X = reinterpret_cast<float *>(ws + L.X);
    float *Hd = reinterpret_cast<float *>(ws + L.H[0]);
    float *Hu = reinterpret_cast<float *>(ws + L.H[1]);
    const StatusSlot status = new_status_slot(g, ws, L);
    s = cuda_status(launch_features(g->host.n, B, w->m, cost, bytes, dev, cur, placed, X, st));
    if (s != PLACETO_OK) return s;
    s = run_embed(g, w, X, B, Hd, Hu, ws, L, flags, st, status, true);
    if (s != PLACETO_OK) return s;
    return run_pool(g, w, X, Hd, Hu, cur, B, logits, probs, ws, L, flags, st, status, true);
}

placeto_status placeto_policy_forward_host(const placeto_graph *g, const placeto_weights *w,
                                           const float *cost, const float *bytes,
                                           const uint8_t *dev, const int32_t *cur,
                                           const uint8_t *placed, int32_t B, float *logits,
                                           float *probs, void *workspace, size_t workspace_bytes,
                                           uint32_t flags, void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s == PLACETO_OK) s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1 || w->m > PLACETO_MAX_M || w->F != w->m + 4) return PLACETO_ERR_INVALID_ARG;
    const Layout L = make_layout(g, w, B, PLACETO_CALL_FORWARD_HOST);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, flags);
    if (s != PLACETO_OK) return s;
    if (!cost || !bytes || !dev || !cur || !placed || !logits) return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t n = (size_t)g->host.n;
    float *d_cost = reinterpret_cast<float *>(ws + L.cost);
    float *d_bytes = reinterpret_cast<float *>(ws + L.bytes);
    uint8_t *d_dev = reinterpret_cast<uint8_t *>(ws + L.dev);
    uint8_t *d_placed = reinterpret_cast<uint8_t *>(ws + L.placed);
    int32_t *d_cur = reinterpret_cast<int32_t *>(ws + L.cur);
    float *d_logits = reinterpret_cast<float *>(ws + L.logits);
    float *d_probs = reinterpret_cast<float *>(ws + L.probs);
    const size_t mB = (size_t)B * w->m * sizeof(float);
    // Page-locked host buffers are addressable from the device: the five inputs are
    // then gathered by one kernel instead of five copies, and the head kernel writes
    // logits and probabilities straight into the caller's buffers. Pageable buffers
    // take the copy path.
    const void *src[5] = {cost, bytes, dev, placed, cur};
    void *dst[5] = {d_cost, d_bytes, d_dev, d_placed, d_cur};
    const size_t len[5] = {n * sizeof(float), n * sizeof(float), n * B, n * B, (size_t)B * sizeof(int32_t)};
    const void *mapped[5];
    bool in_mapped = true;
    for (int i = 0; i < 5 && in_mapped; ++i) in_mapped = (mapped[i] = device_alias(src[i])) != nullptr;
    if (in_mapped) {
        if (launch_stage_inputs(mapped, dst, len, g->info.sm_count, st) != cudaSuccess) return PLACETO_ERR_CUDA;
    } else {
        for (int i = 0; i < 5; ++i)
            if (cudaMemcpyAsync(dst[i], src[i], len[i], cudaMemcpyHostToDevice, st) != cudaSuccess)
                return PLACETO_ERR_CUDA;
    }
    float *out_logits = static_cast<float *>(const_cast<void *>(device_alias(logits)));
    float *out_probs = probs ? static_cast<float *>(const_cast<void *>(device_alias(probs))) : nullptr;
    const bool out_mapped = out_logits && (!probs || out_probs) && aligned16(out_logits) &&
                            (!probs || aligned16(out_probs));
    if (!out_mapped) { out_logits = d_logits; out_probs = probs ? d_probs : nullptr; }
    float *X = reinterpret_cast<float *>(ws + L.X);
    float *Hd = reinterpret_cast<float *>(ws + L.H[0]);
    float *Hu = reinterpret_cast<float *>(ws + L.H[1]);
    // after the gather kernel the whole chain overlaps: the set-up of the message
    // passing kernel (weights, schedule) runs while the inputs cross the host link
    s = cuda_status(launch_features(g->host.n, B, w->m, d_cost, d_bytes, d_dev, d_cur, d_placed, X, st,
                                    in_mapped));
    if (s != PLACETO_OK) return s;
    const StatusSlot status = new_status_slot(g, ws, L);
    s = run_embed(g, w, X, B, Hd, Hu, ws, L, flags, st, status, true);
    if (s != PLACETO_OK) return s;
    s = run_pool(g, w, X, Hd, Hu, d_cur, B, out_logits, out_probs, ws, L, flags, st, status, true);
    if (s != PLACETO_OK) return s;
    if (!out_mapped) {
        if (cudaMemcpyAsync(logits, d_logits, mB, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return PLACETO_ERR_CUDA;
        if (probs && cudaMemcpyAsync(probs, d_probs, mB, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return PLACETO_ERR_CUDA;
    }
    return cuda_status(cudaStreamSynchronize(st));
}

placeto_status placeto_policy_logits_static(const placeto_graph *g, const placeto_weights *w,
                                            const float *X, const float *H_down,
                                            const float *H_up, const int32_t *cur, int32_t B,
                                            float *logits, float *probs, uint32_t flags,
                                            void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1 || !flags_ok(flags) || !on_graph_device(g)) return PLACETO_ERR_INVALID_ARG;
    if ((size_t)B * g->host.n > (size_t)1 << 31) return PLACETO_ERR_UNSUPPORTED;
    const Layout L = make_layout(g, w, B, PLACETO_CALL_LOGITS);   // status record, then the partial sums
    if (L.total > PLACETO_STATIC_SCRATCH_BYTES) return PLACETO_ERR_SCRATCH_LIMIT;
    if (!X || !H_down || !H_up || !cur || !logits) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(H_down) || !aligned16(H_up) || !aligned16(cur) ||
        !aligned16(logits) || (probs && !aligned16(probs)))
        return PLACETO_ERR_INVALID_ARG;
    char *scratch = static_scratch_address(g->device);
    if (!scratch) return PLACETO_ERR_CUDA;
    return run_pool(g, w, X, H_down, H_up, cur, B, logits, probs, scratch, L, flags,
                    static_cast<cudaStream_t>(stream), new_status_slot(g, scratch, L));
}

placeto_status placeto_embed_rounds(const placeto_graph *g, const placeto_weights *w, const float *X,
                                    int32_t B, int32_t rounds, float *H_down, float *H_up,
                                    void *workspace, size_t workspace_bytes, void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1 || rounds < 0) return PLACETO_ERR_INVALID_ARG;
    g->calls.fetch_add(1);
    const Layout L = make_layout(g, w, B, PLACETO_CALL_EMBED_ROUNDS);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, 0);
    if (s != PLACETO_OK) return s;
    if (!X || !H_down || !H_up || !aligned16(X) || !aligned16(H_down) || !aligned16(H_up))
        return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    EmbedArgs a;
    a.lv[0] = g->lv[0]; a.lv[1] = g->lv[1];
    a.f[0] = to_dev(w->f_down); a.f[1] = to_dev(w->f_up);
    a.g[0] = to_dev(w->g_down); a.g[1] = to_dev(w->g_up);
    a.X = X;
    a.H[0] = H_down; a.H[1] = H_up;
    a.M[0] = a.M[1] = nullptr;
    a.n = g->host.n; a.B = B; a.F = w->F; a.d = w->d;
    a.max_level_width = g->host.max_level_width;
    if (rounds == 0) {      // H^0 = 0
        const size_t bytes = (size_t)a.n * B * a.d * sizeof(float);
        if (cudaMemsetAsync(H_down, 0, bytes, st) != cudaSuccess ||
            cudaMemsetAsync(H_up, 0, bytes, st) != cudaSuccess)
            return PLACETO_ERR_CUDA;
        return PLACETO_OK;
    }
    float *msg[4] = {reinterpret_cast<float *>(ws + L.msg[0]), reinterpret_cast<float *>(ws + L.msg_alt[0]),
                     reinterpret_cast<float *>(ws + L.msg[1]), reinterpret_cast<float *>(ws + L.msg_alt[1])};
    return cuda_status(launch_embed_rounds(a, g->info, rounds, msg, st));
}

placeto_status placeto_episode_rollout(const placeto_graph *g, const placeto_weights *w,
                                       const float *cost, const float *bytes,
                                       const int32_t *order, const float *uniforms, int32_t E,
                                       uint8_t *dev, uint8_t *actions, float *logp,
                                       void *workspace, size_t workspace_bytes, uint32_t flags,
                                       void *stream) {
    t_launches = 0;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s == PLACETO_OK) s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (E < 1 || w->m > PLACETO_MAX_M || w->F != w->m + 4) return PLACETO_ERR_INVALID_ARG;
    const Layout L = make_layout(g, w, E, PLACETO_CALL_EPISODE);
    s = common_checks(g, E, workspace, workspace_bytes, L.total, flags);
    if (s != PLACETO_OK) return s;
    if (!cost || !bytes || !order || !dev) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(bytes) || !aligned16(order) || !aligned16(dev) ||
        (uniforms && !aligned16(uniforms)) || (actions && !aligned16(actions)) ||
        (logp && !aligned16(logp)))
        return PLACETO_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *X = reinterpret_cast<float *>(ws + L.X);
    float *Hd = reinterpret_cast<float *>(ws + L.H[0]);
    float *Hu = reinterpret_cast<float *>(ws + L.H[1]);
    EpisodeArgs ep;
    ep.n = g->host.n; ep.E = E; ep.m = w->m;
    ep.order = order; ep.uniforms = uniforms;
    ep.logits = reinterpret_cast<float *>(ws + L.logits);
    ep.dev = dev;
    ep.placed = reinterpret_cast<uint8_t *>(ws + L.placed);
    ep.cur = reinterpret_cast<int32_t *>(ws + L.cur);
    ep.logp = logp; ep.actions = actions;
    float *probs = reinterpret_cast<float *>(ws + L.probs);
    ep.X = X;
    const StatusSlot status = new_status_slot(g, ws, L);

    // Where every kernel of a step takes compact states (the d = 32 sweep and pooling kernels
    // and the fast head kernel), the episodes run without a feature tensor: one byte per (node,
    // episode) is the whole state, and the head kernel makes the transition itself.
    bool compact_path = false;
    if (!(flags & (PLACETO_GENERIC | PLACETO_TENSOR | PLACETO_PER_LEVEL | PLACETO_COOPERATIVE)) && w->m < 63 &&
        L.chunks32 > 0) {
        EmbedArgs ea;
        ea.lv[0] = g->lv[0]; ea.lv[1] = g->lv[1];
        ea.f[0] = to_dev(w->f_down); ea.f[1] = to_dev(w->f_up);
        ea.g[0] = to_dev(w->g_down); ea.g[1] = to_dev(w->g_up);
        ea.n = g->host.n; ea.B = E; ea.F = w->F; ea.d = w->d;
        ea.max_level_width = g->host.max_level_width;
        PoolArgs pa;
        for (int i = 0; i < 3; ++i) { pa.l[i] = to_dev(w->l[i]); pa.h[i] = to_dev(w->h[i]); }
        pa.head = to_dev(w->head);
        pa.n = g->host.n; pa.B = E; pa.F = w->F; pa.d = w->d; pa.m = w->m;
        pa.chunks = L.chunks32; pa.chunk_nodes = L.chunk_nodes32;
        compact_path = embed_d32_fits(ea, g->info) && pool_d32_fits(pa, g->info) && pool_head_takes_compact(pa);
    }
    if (compact_path) {
        CompactState cs;
        cs.cost = cost; cs.bytes = bytes; cs.m = w->m;
        uint8_t *state = reinterpret_cast<uint8_t *>(ws + L.compact);
        cs.state = state;
        cs.cur = ep.cur;
        s = cuda_status(launch_episode_begin_compact(ep.n, E, order, dev, state, ep.cur, st));
        EpisodeStep step;
        step.enabled = 1; step.n = ep.n;
        step.order = order; step.uniforms = uniforms;
        step.state = state; step.cur = ep.cur;
        step.logp = logp; step.actions = actions;
        for (int t = 0; s == PLACETO_OK && t < ep.n; ++t) {
            step.t = t;
            s = run_embed(g, w, nullptr, E, Hd, Hu, ws, L, flags, st, status, true, &cs);
            if (s == PLACETO_OK)
                s = run_pool(g, w, nullptr, Hd, Hu, ep.cur, E, const_cast<float *>(ep.logits), probs, ws, L, flags, st,
                             status, true, &cs, &step);
        }
        if (s == PLACETO_OK) s = cuda_status(launch_episode_end_compact(ep.n, E, state, dev, st));
        return s;
    }
    s = cuda_status(launch_episode_begin(ep, st));
    // the features of the initial states; every later step patches them in place
    if (s == PLACETO_OK)
        s = cuda_status(launch_features(ep.n, E, w->m, cost, bytes, dev, ep.cur, ep.placed, X, st));
    for (int t = 0; s == PLACETO_OK && t < ep.n; ++t) {
        // one policy evaluation of the E current states, then the transition
        s = run_embed(g, w, X, E, Hd, Hu, ws, L, flags, st, status, true);
        if (s == PLACETO_OK)
            s = run_pool(g, w, X, Hd, Hu, ep.cur, E, const_cast<float *>(ep.logits), probs, ws, L, flags, st, status, true);
        if (s == PLACETO_OK) s = cuda_status(launch_episode_step(ep, t, st));
    }
    return s;
}

size_t placeto_simulator_workspace_bytes(const placeto_graph *g, int32_t P, int32_t m) {
    if (!g || P < 1 || m < 1 || m > PLACETO_MAX_M) return 0;
    return sim_workspace_bytes(g->host.n, (int)g->host.n_edges, m, P);
}

placeto_status placeto_simulate_placements(const placeto_graph *g, const float *cost, const float *bytes,
                                           const uint8_t *dev, int32_t P, int32_t m, double bandwidth,
                                           double mem_limit, double mem_scale, double *runtime,
                                           double *peak_memory, double *penalised, void *workspace,
                                           size_t workspace_bytes, void *stream) {
    t_launches = 0;
    if (!g || !g->on_device || P < 1 || m < 1 || m > PLACETO_MAX_M) return PLACETO_ERR_INVALID_ARG;
    if (!(bandwidth > 0.0) || !(mem_scale >= 0.0) || mem_limit != mem_limit || !on_graph_device(g))
        return PLACETO_ERR_INVALID_ARG;
    g->calls.fetch_add(1);
    if (!cost || !bytes || !dev || !workspace || (!runtime && !peak_memory && !penalised)) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(bytes) || !aligned16(dev) || !aligned16(workspace) ||
        (runtime && !aligned16(runtime)) || (peak_memory && !aligned16(peak_memory)) ||
        (penalised && !aligned16(penalised)))
        return PLACETO_ERR_INVALID_ARG;
    if (workspace_bytes < sim_workspace_bytes(g->host.n, (int)g->host.n_edges, m, P))
        return PLACETO_ERR_WORKSPACE;
    SimArgs a;
    a.n = g->host.n; a.n_edges = (int)g->host.n_edges; a.m = m; a.P = P;
    a.child_ptr = g->d_child_ptr; a.child = g->d_child; a.n_parents = g->d_n_parents;
    a.parent_ptr = g->d_parent_ptr; a.parent = g->d_parent;
    a.cost = cost; a.bytes = bytes; a.dev = dev;
    a.bandwidth = bandwidth;
    a.mem_limit = mem_limit; a.mem_scale = mem_scale;
    a.runtime = runtime; a.peak_memory = peak_memory; a.penalised = penalised;
    a.workspace = static_cast<char *>(workspace);
    return cuda_status(launch_simulator(a, static_cast<cudaStream_t>(stream)));
}

placeto_status placeto_simulate_runtime(const placeto_graph *g, const float *cost, const float *bytes,
                                        const uint8_t *dev, int32_t P, int32_t m, double bandwidth,
                                        double *runtime, void *workspace, size_t workspace_bytes,
                                        void *stream) {
    if (!runtime) return PLACETO_ERR_INVALID_ARG;
    return placeto_simulate_placements(g, cost, bytes, dev, P, m, bandwidth, 0.0, 0.0, runtime, nullptr, nullptr,
                                       workspace, workspace_bytes, stream);
}

placeto_status placeto_policy_gradient(const placeto_graph *g, const placeto_weights *w, const float *X,
                                       const float *H_down, const float *H_up, const int32_t *cur,
                                       const int32_t *actions, const float *advantages, float beta,
                                       int32_t B, const placeto_weights *grads, void *workspace,
                                       size_t workspace_bytes, uint32_t flags, void *stream) {
    t_launches = 0;
    if (flags & ~PLACETO_GRAD_ACCUMULATE) return PLACETO_ERR_INVALID_ARG;
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    placeto_status s = embed_weights_ok(w);
    if (s == PLACETO_OK) s = pool_weights_ok(w);
    if (s != PLACETO_OK) return s;
    if (B < 1 || !grads) return PLACETO_ERR_INVALID_ARG;
    g->calls.fetch_add(1);
    // the gradient buffers mirror the weights' shapes
    if (grads->d != w->d || grads->F != w->F || grads->m != w->m) return PLACETO_ERR_INVALID_ARG;
    const placeto_mlp *wn[11] = {&w->f_down, &w->f_up, &w->g_down, &w->g_up, &w->l[0], &w->l[1], &w->l[2],
                                 &w->h[0], &w->h[1], &w->h[2], &w->head};
    const placeto_mlp *gn[11] = {&grads->f_down, &grads->f_up, &grads->g_down, &grads->g_up, &grads->l[0],
                                 &grads->l[1], &grads->l[2], &grads->h[0], &grads->h[1], &grads->h[2],
                                 &grads->head};
    for (int i = 0; i < 11; ++i) {
        if (gn[i]->n_layers != wn[i]->n_layers || gn[i]->in_dim != wn[i]->in_dim ||
            gn[i]->out_dim != wn[i]->out_dim ||
            (wn[i]->n_layers == 2 && gn[i]->hidden_dim != wn[i]->hidden_dim))
            return PLACETO_ERR_INVALID_ARG;
        if (!gn[i]->W1 || !gn[i]->b1 || !aligned16(gn[i]->W1) || !aligned16(gn[i]->b1)) return PLACETO_ERR_INVALID_ARG;
        if (wn[i]->n_layers == 2 && (!gn[i]->W2 || !gn[i]->b2 || !aligned16(gn[i]->W2) || !aligned16(gn[i]->b2)))
            return PLACETO_ERR_INVALID_ARG;
    }
    const Layout L = make_layout(g, w, B, PLACETO_CALL_GRADIENT);
    s = common_checks(g, B, workspace, workspace_bytes, L.total, 0);
    if (s != PLACETO_OK) return s;
    if (!X || !H_down || !H_up || !cur || !actions || !advantages) return PLACETO_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(H_down) || !aligned16(H_up) || !aligned16(cur) ||
        !aligned16(actions) || !aligned16(advantages))
        return PLACETO_ERR_INVALID_ARG;
    GradArgs a{};
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    a.n = g->host.n; a.B = B; a.d = w->d; a.F = w->F; a.m = w->m;
    a.relation = g->d_relation;
    a.lv[0] = g->lv[0]; a.lv[1] = g->lv[1];
    a.child_ptr = g->d_child_ptr; a.child = g->d_child;
    a.parent_ptr = g->d_parent_ptr; a.parent = g->d_parent;
    a.f[0] = to_dev(w->f_down); a.f[1] = to_dev(w->f_up);
    a.g[0] = to_dev(w->g_down); a.g[1] = to_dev(w->g_up);
    for (int i = 0; i < 3; ++i) { a.l[i] = to_dev(w->l[i]); a.h[i] = to_dev(w->h[i]); }
    a.head = to_dev(w->head);
    // The paper's own f and g are single layers (Appendix A.7). y = relu(W x + b) is, bit for
    // bit, the two-layer network relu(I relu(W x + b) + 0): the second ReLU sees values >= 0.
    // The kernels differentiate that form; its identity layer lives in the workspace and the
    // gradient of the identity is written to scratch beside it and dropped.
    float *extra = reinterpret_cast<float *>(ws + L.grad_extra);
    const size_t dd = (size_t)w->d * w->d, one = dd + w->d;
    DevMlp *mp[4] = {&a.f[0], &a.f[1], &a.g[0], &a.g[1]};
    bool widened[4] = {false, false, false, false};
    for (int k = 0; k < 4; ++k) {
        DevMlp &net = *mp[k];
        if (net.n_layers != 1 || net.act != 0 || net.final_act != 1) continue;
        float *eye = extra + (size_t)k * 2 * one;
        if (launch_identity_layer(eye, w->d, st) != cudaSuccess) return PLACETO_ERR_CUDA;
        net.n_layers = 2;
        net.hidden_dim = net.out_dim;
        net.W2 = eye;
        net.b2 = eye + dd;
        widened[k] = true;
    }
    if (!policy_gradient_applicable(a)) return PLACETO_ERR_UNSUPPORTED;
    a.X = X; a.H[0] = H_down; a.H[1] = H_up;
    a.cur = cur; a.actions = actions; a.advantages = advantages; a.beta = beta;
    a.accumulate = (flags & PLACETO_GRAD_ACCUMULATE) ? 1 : 0;
    auto out = [](const placeto_mlp &m) {
        GradOut o;
        o.W1 = const_cast<float *>(m.W1); o.b1 = const_cast<float *>(m.b1);
        o.W2 = const_cast<float *>(m.W2); o.b2 = const_cast<float *>(m.b2);
        return o;
    };
    a.gf[0] = out(grads->f_down); a.gf[1] = out(grads->f_up);
    a.gg[0] = out(grads->g_down); a.gg[1] = out(grads->g_up);
    for (int i = 0; i < 3; ++i) { a.gl[i] = out(grads->l[i]); a.gh[i] = out(grads->h[i]); }
    a.ghead = out(grads->head);
    GradOut *gp[4] = {&a.gf[0], &a.gf[1], &a.gg[0], &a.gg[1]};
    for (int k = 0; k < 4; ++k)
        if (widened[k]) {
            gp[k]->W2 = extra + (size_t)k * 2 * one + one;
            gp[k]->b2 = gp[k]->W2 + dd;
        }
    return cuda_status(launch_policy_gradient(a, g->info, reinterpret_cast<float *>(ws + L.grad), st));
}

placeto_status placeto_simple_aggregator(const placeto_graph *g, const placeto_aggregator_weights *w,
                                         const float *X, int32_t B, float *logits, float *probs, void *stream) {
    t_launches = 0;
    if (!g || !g->on_device || !w || B < 1 || !on_graph_device(g)) return PLACETO_ERR_INVALID_ARG;
    g->calls.fetch_add(1);
    if (w->d < 1 || w->F < 1 || w->m < 1) return PLACETO_ERR_INVALID_ARG;
    if (w->d > PLACETO_MAX_D || w->F > PLACETO_MAX_F || w->m > PLACETO_MAX_M + 4) return PLACETO_ERR_UNSUPPORTED;
    if (!mlp_ok(w->l, w->F, w->d) || !mlp_ok(w->h, w->d, w->d) || !mlp_ok(w->head, w->d, w->m))
        return PLACETO_ERR_INVALID_ARG;
    if ((size_t)B * g->host.n > (size_t)1 << 31) return PLACETO_ERR_UNSUPPORTED;
    if (!X || !logits || !aligned16(X) || !aligned16(logits) || (probs && !aligned16(probs)))
        return PLACETO_ERR_INVALID_ARG;
    const cudaError_t e = launch_simple_aggregator(to_dev(w->l), to_dev(w->h), to_dev(w->head), X, g->host.n, B, w->F,
                                                   w->d, w->m, logits, probs, g->info,
                                                   static_cast<cudaStream_t>(stream));
    return e == cudaErrorNotSupported ? PLACETO_ERR_UNSUPPORTED : cuda_status(e);
}

placeto_status placeto_last_status(const placeto_graph *g, const void *workspace, void *stream) {
    if (!g || !g->on_device) return PLACETO_ERR_INVALID_ARG;
    const char *at = static_cast<const char *>(workspace);
    if (!at) {
        at = static_scratch_address(g->device);
        if (!at) return PLACETO_ERR_CUDA;
    }
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PLACETO_ERR_CUDA;
    int rec[4] = {0, 0, 0, 0};
    if (cudaMemcpy(rec, at, sizeof(rec), cudaMemcpyDeviceToHost) != cudaSuccess) return PLACETO_ERR_CUDA;
    if (rec[0] != kStatusMagic0 || rec[1] != kStatusMagic1 || rec[2] != g->calls.load()) return PLACETO_OK;
    return rec[3] > 0 && rec[3] <= PLACETO_ERR_TIMEOUT ? static_cast<placeto_status>(rec[3]) : PLACETO_ERR_CUDA;
}

placeto_status placeto_debug_wait_timeout(const placeto_graph *g, void *workspace, size_t workspace_bytes,
                                          void *stream) {
    t_launches = 0;
    if (!g || !g->on_device || !workspace || !aligned16(workspace)) return PLACETO_ERR_INVALID_ARG;
    if (!on_graph_device(g)) return PLACETO_ERR_INVALID_ARG;
    if (workspace_bytes < kStatusBytes) return PLACETO_ERR_WORKSPACE;
    Layout L{};
    return cuda_status(launch_wait_timeout_probe(new_status_slot(g, static_cast<char *>(workspace), L),
                                                 static_cast<cudaStream_t>(stream)));
}

int32_t placeto_last_launch_count(void) { return t_launches; }

}  // extern "C"
