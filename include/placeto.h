/*
 * placeto.h - C ABI of the B200 (sm_100a) library for the Placeto policy forward.
 *
 * The library evaluates, for one computation DAG and a batch of B placement
 * states, the graph-embedding policy network of Placeto (arXiv 1906.08879,
 * Sec. 2.2 and Appendix A.7):
 *
 *   step 1  raw features per node and state                (Sec. 2.1, Sec. 2.2 step 1)
 *   step 2  top-down and bottom-up message passing,
 *           h_v = g( sum_{u in nbr(v)} f([h_u || x_u]) )    (Sec. 2.2 step 2)
 *   step 3  pooling over the nodes that can reach the current node, that it
 *           can reach, and the rest: h_i( sum l_i(e_u) )    (Sec. 2.2 step 3)
 *   head    two-layer feed-forward net + softmax over the m devices (Appendix A.7)
 *
 * Conventions
 *   - Pointers are marked HOST or DEVICE. All DEVICE pointers must be 16-byte
 *     aligned and belong to the device that was current at placeto_graph_create;
 *     that device must be current again at every call (PLACETO_ERR_INVALID_ARG
 *     otherwise).
 *   - The caller owns every buffer (inputs, outputs, weights, workspace); the
 *     library owns only placeto_graph objects. Forward calls allocate nothing,
 *     do not synchronise (except the _host variant, see there) and run
 *     asynchronously on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream). Two calls may run concurrently if their workspaces and
 *     outputs are distinct.
 *   - Every call returns a placeto_status. Problems the host can see (null or
 *     misaligned pointers, sizes out of range, networks whose dimensions do not
 *     fit d, F, m, a workspace that is too small, a graph with a cycle) are
 *     rejected before any launch and leave the outputs untouched. CUDA launch
 *     failures map to PLACETO_ERR_CUDA. Nothing aborts or traps.
 *   - Node ids in all tensors are the caller's ids. Layouts are row-major:
 *     X[n][B][F], H[n][B][d], logits/probs[B][m], dev/placed[B][n].
 *   - Arithmetic is fp32. The order of the sums over neighbours and sets is
 *     unspecified but fixed: a call is run-to-run deterministic for fixed
 *     arguments and flags.
 */
#ifndef PLACETO_H_
#define PLACETO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PLACETO_OK = 0,
    PLACETO_ERR_INVALID_ARG = 1, /* null/misaligned pointer, size or dimension out of range */
    PLACETO_ERR_NOT_DAG = 2,     /* cycle, self-loop or node id out of range */
    PLACETO_ERR_WORKSPACE = 3,   /* workspace smaller than placeto_workspace_bytes() */
    PLACETO_ERR_UNSUPPORTED = 4, /* dimensions beyond the limits below, or flag not applicable */
    PLACETO_ERR_CUDA = 5,        /* a CUDA runtime call or launch failed */
    PLACETO_ERR_NO_MEMORY = 6,   /* host or device allocation failed in graph_create */
    PLACETO_ERR_SCRATCH_LIMIT = 7,/* batch too large for the built-in scratch of
                                     placeto_policy_logits_static */
    PLACETO_ERR_TIMEOUT = 8      /* a bounded wait inside a kernel ran out (reported through the
                                     status word, see placeto_last_status) */
} placeto_status;

/* Limits of the library. */
#define PLACETO_MAX_D 128      /* embedding width d */
#define PLACETO_MAX_F 64       /* feature width F */
#define PLACETO_MAX_M 60       /* devices m (F = m + 4 in build_features) */
#define PLACETO_MAX_HIDDEN 1024/* hidden width of any network */
#define PLACETO_MAX_NODES 16384

/* Human-readable name of a status (static string, never NULL). */
const char *placeto_status_string(placeto_status s);

/* ------------------------------------------------------------------ graph -- */

typedef struct placeto_graph placeto_graph; /* opaque, library-owned */

/* placeto_graph_create flags */
#define PLACETO_GRAPH_DEVICE 0u    /* build on the host and upload to the current device */
#define PLACETO_GRAPH_HOST_ONLY 1u /* build the host plan only (no CUDA call; forward calls
                                      on such a graph return PLACETO_ERR_INVALID_ARG) */

/*
 * Builds the static plan of a DAG G(V, E) (Sec. 2: nodes are op groups, edges
 * data dependencies u -> v) from a HOST edge list in any order:
 *   - checks ids and acyclicity (PLACETO_ERR_NOT_DAG), drops repeated edges
 *     (neighbours are sets);
 *   - top-down levels (longest path from a root) and bottom-up levels (longest
 *     path to a leaf), nodes bucketed by level, with the parent (resp. child)
 *     lists in CSR form in level order: the schedule of step 2;
 *   - the relation of every pair (c, u): u can reach c / c can reach u /
 *     neither / same node: the three sets of step 3.
 * src, dst: HOST int32[n_edges] (may be NULL when n_edges == 0). n >= 1.
 * On success *out owns host and (unless HOST_ONLY) device copies of the plan;
 * release it with placeto_graph_destroy. On failure *out is NULL.
 */
placeto_status placeto_graph_create(int32_t n, int64_t n_edges, const int32_t *src,
                                    const int32_t *dst, uint32_t flags, placeto_graph **out);

/* Sizes of the plan. Any output pointer may be NULL. n_edges counts distinct edges. */
placeto_status placeto_graph_info(const placeto_graph *g, int32_t *n, int64_t *n_edges,
                                  int32_t *n_levels_down, int32_t *n_levels_up,
                                  int32_t *max_level_width);

/*
 * Read-only HOST view of the plan, valid until placeto_graph_destroy; meant
 * for inspection and tests. dir 0 = top-down (neighbours are parents), 1 =
 * bottom-up (neighbours are children).
 *   level_ptr[n_levels+1] : positions of each level's nodes in `order`
 *   order[n]              : node ids sorted by level, ascending id inside a level
 *   nbr_ptr[n+1], nbr[]   : neighbour ids of order[p] are nbr[nbr_ptr[p] .. nbr_ptr[p+1]), ascending
 *   n_slots, own_slot[n], nbr_slot[] : on-chip message slots. The message of order[p] is kept
 *                           in slot own_slot[p] (-1 if no node consumes it) from its level until
 *                           the last level that reads it; nbr_slot[e] is the slot of nbr[e].
 *                           Slots are shared by nodes whose lifetimes do not overlap.
 *   relation[n*n]         : relation[c*n+u] = 0 u can reach c, 1 c can reach u, 2 neither, 3 u == c
 */
typedef struct {
    int32_t n_levels;
    const int32_t *level_ptr, *order, *nbr_ptr, *nbr;
    int32_t n_slots;
    const int32_t *own_slot, *nbr_slot;
} placeto_level_view;
placeto_status placeto_graph_host_view(const placeto_graph *g, placeto_level_view *down,
                                       placeto_level_view *up, const uint8_t **relation);

/* Releases the plan (device memory is freed with the creating device current). NULL is a no-op. */
void placeto_graph_destroy(placeto_graph *g);

/* ---------------------------------------------------------------- weights -- */

/* One feed-forward network (Appendix A.7): y = act(v W1 + b1), then for two
 * layers y = y W2 + b2; the activation also follows the last layer when
 * final_act is 1. W row-major [in][out]. Pointers are DEVICE float arrays
 * (W2, b2 NULL for one layer). */
typedef struct {
    int32_t n_layers;                     /* 1 or 2 */
    int32_t in_dim, hidden_dim, out_dim;  /* hidden_dim ignored for one layer */
    const float *W1, *b1, *W2, *b2;
    int32_t act;                          /* 0 relu, 1 identity */
    int32_t final_act;                    /* 0 or 1 */
} placeto_mlp;

/* All networks of the policy. f: (d+F) -> d and g: d -> d per direction
 * (separate parameters, shared by all nodes of the direction); l[i]: (2d+F) -> d
 * and h[i]: d -> d for i = 0 parents set, 1 children set, 2 parallel set;
 * head: (5d+F) -> hidden -> m, normally with final_act = 0. */
typedef struct {
    int32_t d, F, m;
    placeto_mlp f_down, g_down, f_up, g_up;
    placeto_mlp l[3], h[3];
    placeto_mlp head;
} placeto_weights;

/* ------------------------------------------------------------------ calls -- */

/* Schedule of step 2 (the result does not depend on it beyond rounding order). */
#define PLACETO_AUTO 0u        /* library picks */
#define PLACETO_PER_LEVEL 1u   /* one launch per topological level */
#define PLACETO_SLICED 2u      /* persistent: each thread block owns a slice of the state batch
                                  and walks all levels, synchronising only inside the block
                                  (states never interact) */
#define PLACETO_COOPERATIVE 4u /* persistent cooperative launch: a level's nodes are spread over
                                  blocks, grid-wide sync between levels (small B, wide levels) */
#define PLACETO_GENERIC 8u     /* use only the dimension-generic kernels (no specialised ones) */
#define PLACETO_FMA_ONLY 16u   /* keep step 2 on the FP32 FMA pipes: do not use the tensor-core
                                  kernel (TF32 head + tail split, three products per step) that
                                  d = 64 otherwise takes */
#define PLACETO_TENSOR 32u     /* use the tensor-core kernel of step 2 that gives every block whole 16-row
                                  tiles (all warps on one layer at a time) wherever it applies (d = 32 or
                                  64); the library itself picks other kernels there */
#define PLACETO_TCGEN05 64u    /* d = 64: take the kernel built on tcgen05.mma with accumulators in tensor
                                  memory instead of the warp-level (mma.sync) tensor-core kernel that is
                                  the default there (measured slower at the configured batch sizes) */
#define PLACETO_PIPELINE 128u  /* d = 64: take the kernel that runs the four layers of g and f as a pipeline
                                  (a group of warps per layer, tiles of eight rows). It is what the
                                  library picks at d = 64 anyway; the flag pins the choice. */

typedef enum {
    PLACETO_CALL_EMBED = 0,       /* placeto_embed_forward */
    PLACETO_CALL_LOGITS = 1,      /* placeto_policy_logits */
    PLACETO_CALL_FORWARD = 2,     /* placeto_policy_forward */
    PLACETO_CALL_FORWARD_HOST = 3,/* placeto_policy_forward_host */
    PLACETO_CALL_EPISODE = 4,     /* placeto_episode_rollout (B = number of episodes) */
    PLACETO_CALL_EMBED_ROUNDS = 5,/* placeto_embed_rounds */
    PLACETO_CALL_GRADIENT = 6     /* placeto_policy_gradient */
} placeto_call;

/* Bytes of DEVICE workspace `call` needs for batch size B (0 on invalid arguments).
 * The workspace holds the per-node messages of step 2, partial sums of step 3 and,
 * for the two policy_forward calls, the intermediate tensors X, H_down, H_up
 * (plus the staged inputs and results for the _host call). */
size_t placeto_workspace_bytes(const placeto_graph *g, const placeto_weights *w, int32_t B,
                               placeto_call call, uint32_t flags);

/*
 * Step 1 (Sec. 2.1; Sec. 2.2 step 1): X[v][b] = [cost_v, bytes_v, one-hot_m(dev[b][v]),
 * 1[v == cur[b]], placed[b][v] != 0], F = m + 4.
 * cost, bytes: DEVICE float[n]; dev, placed: DEVICE uint8[B][n] (dev values < m; a larger
 * value yields an all-zero one-hot); cur: DEVICE int32[B]; X: DEVICE float[n][B][m+4] (out).
 */
placeto_status placeto_build_features(const placeto_graph *g, const float *cost,
                                      const float *bytes, const uint8_t *dev, const int32_t *cur,
                                      const uint8_t *placed, int32_t m, int32_t B, float *X,
                                      void *stream);

/*
 * Step 2 (Sec. 2.2 step 2), one progressive sweep per direction in topological
 * order: h_v = g( sum_{u in nbr(v)} f([h_u || x_u]) ), nbr = parents for H_down,
 * children for H_up; an empty neighbour set sums to zero. Uses w->f_*, w->g_*, w->d, w->F.
 * X: DEVICE float[n][B][F] (in); H_down, H_up: DEVICE float[n][B][d] (out).
 * workspace: DEVICE, at least placeto_workspace_bytes(.., PLACETO_CALL_EMBED, flags).
 */
placeto_status placeto_embed_forward(const placeto_graph *g, const placeto_weights *w,
                                     const float *X, int32_t B, float *H_down, float *H_up,
                                     void *workspace, size_t workspace_bytes, uint32_t flags,
                                     void *stream);

/*
 * Step 3 and the head (Sec. 2.2 step 3, Appendix A.7). With e_u = [h_down_u || h_up_u || x_u]
 * and c = cur[b]: a_i = h_i( sum_{u in S_i(c)} l_i(e_u) ) for the three sets (an empty set
 * sums to zero), z = [e_c || a_0 || a_1 || a_2], logits = head(z), probs = softmax(logits)
 * (max-subtracted). cur is authoritative for the sets; it is not re-derived from X.
 * cur: DEVICE int32[B], each in [0, n) (a value out of range makes that state's outputs NaN);
 * logits: DEVICE float[B][m] (out); probs: DEVICE float[B][m] (out) or NULL.
 */
placeto_status placeto_policy_logits(const placeto_graph *g, const placeto_weights *w,
                                     const float *X, const float *H_down, const float *H_up,
                                     const int32_t *cur, int32_t B, float *logits, float *probs,
                                     void *workspace, size_t workspace_bytes, uint32_t flags,
                                     void *stream);

/*
 * Whole path on DEVICE state arrays: steps 1-3 and the head; X and H live in the
 * workspace. Arguments as in placeto_build_features and placeto_policy_logits
 * (w->F must equal w->m + 4).
 */
placeto_status placeto_policy_forward(const placeto_graph *g, const placeto_weights *w,
                                      const float *cost, const float *bytes, const uint8_t *dev,
                                      const int32_t *cur, const uint8_t *placed, int32_t B,
                                      float *logits, float *probs, void *workspace,
                                      size_t workspace_bytes, uint32_t flags, void *stream);

/*
 * Whole path from HOST state arrays to HOST results: brings cost, bytes, dev, cur,
 * placed to the device, runs the path, returns logits (and probs unless NULL) to the
 * host and waits for the stream before returning. When all five inputs are page-locked
 * host memory (cudaHostAlloc, cudaHostRegister, a pinned torch tensor) one kernel
 * gathers them across the host link, and when the outputs are page-locked too the
 * head kernel writes them in place; pageable buffers are moved with cudaMemcpyAsync
 * on `stream` instead. Either way the same bytes cross the link once per call.
 * Weights and workspace stay DEVICE pointers.
 */
placeto_status placeto_policy_forward_host(const placeto_graph *g, const placeto_weights *w,
                                           const float *cost, const float *bytes,
                                           const uint8_t *dev, const int32_t *cur,
                                           const uint8_t *placed, int32_t B, float *logits,
                                           float *probs, void *workspace, size_t workspace_bytes,
                                           uint32_t flags, void *stream);

/*
 * Step 2 in the synchronous form the paper states (Sec. 2.2 step 2: the message
 * passing updates are repeated k times, k a hyper-parameter): H^0 = 0 and, for
 * r = 1 .. rounds, every node at once from the previous round's values,
 *   H^r_v = g( sum_{u in nbr(v)} f([H^(r-1)_u || x_u]) ),
 * top-down over parents into H_down and bottom-up over children into H_up, each
 * with its own f and g. Output: H^rounds. For rounds >= depth of the graph the
 * result equals placeto_embed_forward's (the progressive sweep is its fixed
 * point); fewer rounds give the truncated, local summaries. rounds + 1 launches
 * of the dimension-generic kernel; every width, depth and activation is accepted.
 * X, H_down, H_up, B as for placeto_embed_forward; rounds >= 0 (0 gives zeros).
 * workspace: DEVICE, at least placeto_workspace_bytes(.., PLACETO_CALL_EMBED_ROUNDS, 0).
 */
placeto_status placeto_embed_rounds(const placeto_graph *g, const placeto_weights *w, const float *X,
                                    int32_t B, int32_t rounds, float *H_down, float *H_up,
                                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * A whole placement episode per call, for E independent episodes on one graph
 * (the MDP of Sec. 2.1 of the paper driven by the policy of Sec. 2.2): for
 * t = 0 .. n-1 the node order[t] is current; the policy is evaluated on the E
 * current states (features, both passes, pooling, head: the same kernels as
 * placeto_policy_forward); every episode picks a device for its current node;
 * the node takes that device and is marked visited. Visited flags start at 0 and
 * the current node itself counts as not yet visited. All steps are queued on
 * `stream` without a host round trip: n * (policy kernels + one transition kernel).
 * The feature tensor is built once; a transition patches the two rows it changes.
 *
 * cost, bytes : DEVICE float[n].
 * order       : DEVICE int32[n], the visiting order, a permutation of 0 .. n-1 (the
 *               paper leaves the order arbitrary). Not checked: an id outside
 *               [0, n) makes that step's policy output NaN and leaves the
 *               placement untouched; a repeated id is visited twice.
 * uniforms    : NULL for greedy episodes (largest logit, lowest device among equals),
 *               else DEVICE float[E][n] of numbers in [0, 1): step t of episode e takes
 *               the first device k with p_0 + .. + p_k > uniforms[e][t], p = softmax(logits).
 * dev         : DEVICE uint8[E][n], in: the initial placement (devices < m); out: the
 *               final one (every node carries the device chosen at its step).
 * actions     : DEVICE uint8[E][n] or NULL, the device chosen at step t (by step, not by node).
 * logp        : DEVICE float[E][n] or NULL, log pi(action | state) of step t.
 * workspace   : DEVICE, at least placeto_workspace_bytes(g, w, E, PLACETO_CALL_EPISODE, flags).
 * Requires w->F == w->m + 4. Errors as for placeto_policy_forward.
 */
placeto_status placeto_episode_rollout(const placeto_graph *g, const placeto_weights *w,
                                       const float *cost, const float *bytes,
                                       const int32_t *order, const float *uniforms, int32_t E,
                                       uint8_t *dev, uint8_t *actions, float *logp,
                                       void *workspace, size_t workspace_bytes, uint32_t flags,
                                       void *stream);

/*
 * Simulated run time of P placements of the graph under the event-based execution
 * model of the paper's simulator (Appendix A.5): one operation at a time per
 * device, taken from a FIFO queue of runnable operations; one output tensor at a
 * time per device bus, overlapping with compute; an operation becomes runnable when
 * all parents have finished and their outputs have arrived on its device; an
 * operation takes cost[v], a transfer bytes[u] / bandwidth; the result is the time
 * stamp of the last operation to finish. One thread simulates one placement.
 * Readings where the paper is silent: one run time per operation whatever the
 * device; a tensor is sent once to each distinct device that hosts a child; a free
 * device or bus starts the head of its queue at once; equal time stamps are handled
 * in the order the events were created.
 *
 * cost, bytes : DEVICE float[n].          dev : DEVICE uint8[P][n], devices < m.
 * bandwidth   : > 0, in units of bytes[] per unit of cost[].
 * runtime     : DEVICE double[P]; NaN for a placement that names a device >= m.
 * workspace   : DEVICE, at least placeto_simulator_workspace_bytes(g, P, m).
 * Times are IEEE doubles added and divided in the model's order: reproducible.
 */
size_t placeto_simulator_workspace_bytes(const placeto_graph *g, int32_t P, int32_t m);
placeto_status placeto_simulate_runtime(const placeto_graph *g, const float *cost, const float *bytes,
                                        const uint8_t *dev, int32_t P, int32_t m, double bandwidth,
                                        double *runtime, void *workspace, size_t workspace_bytes,
                                        void *stream);

/*
 * The same simulation with the devices' peak memory and the memory-penalised run time
 * (Appendix A.5: the operations' start and end time stamps together with the tensor sizes
 * predict the peak memory utilisation of the devices; Appendix A.7: R(p) = r if m <= M,
 * r + c (m - M) otherwise, m the largest peak over the devices, M the memory limit, c a
 * scale factor, 2 in the paper's experiments).
 * Reading taken for the release of tensors, which the paper leaves open: a copy of an
 * operation's output occupies the producer's device from the START of the producer until
 * every child placed there has finished and every transfer of it to another device is done;
 * it occupies another device from the START of the transfer there until every child placed
 * there has finished; the output of an operation without children is never released.
 *
 * mem_limit, mem_scale : M and c, in the units of bytes[] and of cost[] per unit of bytes[].
 * runtime     : DEVICE double[P] or NULL.       peak_memory : DEVICE double[P][m] or NULL.
 * penalised   : DEVICE double[P] or NULL, R(p). At least one of the three must be given.
 * Everything else as for placeto_simulate_runtime (same workspace size, NaN for a
 * placement that names a device >= m, bit-reproducible sums).
 */
placeto_status placeto_simulate_placements(const placeto_graph *g, const float *cost, const float *bytes,
                                           const uint8_t *dev, int32_t P, int32_t m, double bandwidth,
                                           double mem_limit, double mem_scale, double *runtime,
                                           double *peak_memory, double *penalised, void *workspace,
                                           size_t workspace_bytes, void *stream);

/*
 * Gradient of the training objective with respect to every weight and bias of the
 * policy, for a batch of B states (Appendix A.1 of the paper: REINFORCE,
 * sum_b grad log pi(a_b | s_b) * A_b with A_b = return minus baseline; Appendix A.7:
 * an entropy term that encourages exploration):
 *     J = sum_b advantages[b] * log pi(actions[b] | s_b) + beta * sum_b H(pi(. | s_b)),
 *     H(p) = - sum_k p_k log p_k.
 * Reverse-mode differentiation of the forward path: the head and the pooling per
 * state, the two message-passing sweeps level by level in reverse, then every
 * layer's dW = in^T dpre, db = sum dpre as chunked sums added in a fixed order (no
 * atomics: reproducible bit for bit).
 *
 * X, H_down, H_up : DEVICE, as produced by placeto_build_features / placeto_embed_forward
 *                   for the same states and weights.
 * cur, actions    : DEVICE int32[B] (actions < m; a state whose cur is outside [0, n)
 *                   contributes nothing).      advantages : DEVICE float[B].
 * grads           : a placeto_weights of the same shapes as w whose pointers address
 *                   writable DEVICE buffers; every array is overwritten with dJ/d(array), or,
 *                   with PLACETO_GRAD_ACCUMULATE in flags, has dJ/d(array) added to it (a large
 *                   set of states can then be differentiated in several calls).
 * workspace       : DEVICE, at least placeto_workspace_bytes(.., PLACETO_CALL_GRADIENT, 0):
 *                   about 2 * n * B * (2 * (hidden_f + hidden_g) + 6 d) + 3 n B d floats.
 * Shapes: ReLU f and g of one layer (the paper's own, Appendix A.7) or two, single-layer
 * ReLU l_i and h_i, two-layer head with a ReLU hidden layer and a linear output; otherwise
 * PLACETO_ERR_UNSUPPORTED. A single-layer f or g is differentiated as the two-layer network
 * relu(I relu(W x + b) + 0) that it equals bit for bit.
 */
#define PLACETO_GRAD_ACCUMULATE 1u
placeto_status placeto_policy_gradient(const placeto_graph *g, const placeto_weights *w, const float *X,
                                       const float *H_down, const float *H_up, const int32_t *cur,
                                       const int32_t *actions, const float *advantages, float beta,
                                       int32_t B, const placeto_weights *grads, void *workspace,
                                       size_t workspace_bytes, uint32_t flags, void *stream);

/*
 * placeto_policy_logits without a workspace argument, for callers that must not
 * allocate device memory. (The paper has no counterpart: this is a deployment
 * variant of the call above, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving
 * loop with a frozen memory budget, in a plug-in whose host application owns the
 * allocator, or in a process that must not trigger the implicit device
 * synchronisation that an allocation causes. Such a caller still passes every
 * input and output buffer (X, H_down, H_up, cur, logits, probs), exactly as for
 * placeto_policy_logits; only the chunk partial sums of step 3, which the normal
 * call keeps in the caller's workspace, live instead in an array that is part of
 * the library image: PLACETO_STATIC_SCRATCH_BYTES bytes of device memory on every
 * GPU that loads the library, held until the process exits.
 *
 * Limits and rules
 *   - The partial sums need chunks * B * 3 * d floats (chunks grows with n). If that
 *     exceeds PLACETO_STATIC_SCRATCH_BYTES the call returns PLACETO_ERR_SCRATCH_LIMIT
 *     and launches nothing; use placeto_policy_logits with a workspace then.
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating
 *     library routine. The first call on each device looks up the array's device
 *     address (a one-time set-up); make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left there. Nothing in it has to start at zero: each call writes every
 *     entry before reading it. Two calls that overlap on the GPU (different streams,
 *     or different host threads) would overwrite each other's sums: serialise them.
 *   - Results are identical to placeto_policy_logits for the same arguments and flags.
 */
#define PLACETO_STATIC_SCRATCH_BYTES (4u << 20)
placeto_status placeto_policy_logits_static(const placeto_graph *g, const placeto_weights *w,
                                            const float *X, const float *H_down,
                                            const float *H_up, const int32_t *cur, int32_t B,
                                            float *logits, float *probs, uint32_t flags,
                                            void *stream);

/*
 * The "simple aggregator" policy of the paper's ablation (Sec. 4.3, "Alternative policy
 * architectures", variant 1: one feed-forward network aggregates all the node features of
 * the graph, another one with softmax outputs predicts the placement): no message passing,
 * no sets. Reading taken (the paper gives no formula): the aggregate is the sum over ALL
 * nodes of a per-node network, squashed as the pooling summaries of Sec. 2.2 step 3 are,
 *     a = h( sum_{u in V} l(x_u) ),   logits = head(a),   probs = softmax(logits);
 * the current node is in the sum like every other node and is told apart by its
 * is-current feature alone. (The other ablation, the "simple partitioner", needs no entry
 * point: it is placeto_policy_logits on embeddings of zero.)
 *   w      : l: F -> d, h: d -> d, head: d -> hidden -> m (one or two layers each).
 *   X      : DEVICE float[n][B][F] as built by placeto_build_features.
 *   logits : DEVICE float[B][m] (out); probs: DEVICE float[B][m] (out) or NULL.
 * One launch, no workspace; sums run in a fixed order (reproducible).
 */
typedef struct {
    int32_t d, F, m;
    placeto_mlp l, h, head;
} placeto_aggregator_weights;
placeto_status placeto_simple_aggregator(const placeto_graph *g, const placeto_aggregator_weights *w,
                                         const float *X, int32_t B, float *logits, float *probs, void *stream);

/*
 * What the kernels of the most recent call on `g` reported, read back after `stream` has
 * drained (this call synchronises it). The library's kernels never wait without a limit: a
 * wait on an asynchronous copy or on another warp that runs out makes the kernel leave, turn
 * the affected outputs into NaN and write a 16-byte record into the first bytes of the call's
 * workspace (the first 256 bytes of every workspace are reserved for it); a library built with
 * -DPLACETO_DEBUG also records indices that its kernels found out of range (reported as
 * PLACETO_ERR_INVALID_ARG; those accesses are skipped, nothing traps). The record carries the
 * number of the call that wrote it, so nothing has to be cleared between calls and the
 * contents of a fresh workspace cannot be mistaken for a report.
 *   workspace : the workspace of that call, or NULL after placeto_policy_logits_static
 *               (its record sits at the start of the built-in scratch).
 * Returns PLACETO_OK, PLACETO_ERR_TIMEOUT, PLACETO_ERR_INVALID_ARG (debug build) or
 * PLACETO_ERR_CUDA (the read itself failed). Calls on one graph object from several host
 * threads share the call counter: ask before the next call is issued.
 */
placeto_status placeto_last_status(const placeto_graph *g, const void *workspace, void *stream);

/*
 * Runs the time-out path on purpose, for tests of the error channel (the paper has no
 * counterpart): one tiny kernel announces more bytes to a barrier than its copy delivers,
 * polls a few thousand times and gives up exactly as the library's kernels would, reporting
 * PLACETO_ERR_TIMEOUT to placeto_last_status. Nothing faults, traps or hangs; the device stays
 * usable. workspace: DEVICE, at least 256 bytes.
 */
placeto_status placeto_debug_wait_timeout(const placeto_graph *g, void *workspace, size_t workspace_bytes,
                                          void *stream);

/* Number of kernels the most recent forward call of this thread launched (for accounting). */
int32_t placeto_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PLACETO_H_ */
