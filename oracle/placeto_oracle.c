/*
 * CPU checker for the Placeto policy forward (test infrastructure only).
 *
 * A plain, slow evaluation of what the policy network computes for a batch of
 * placement states on one DAG, in double precision (or in single precision
 * when compiled with -DORACLE_REAL=float, as a rounding canary). It is written
 * from the paper's definitions and shares nothing with the CUDA library; only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Paper passages followed:
 *   raw features ................ Sec. 2.1 (state) and Sec. 2.2 step 1
 *   message passing ............. Sec. 2.2 step 2: x_v <- g(sum_{u in xi(v)} f(x_u)),
 *                                 top-down (xi = parents) and bottom-up (xi = children),
 *                                 separate parameters, shared by all nodes of a direction
 *   group pooling ............... Sec. 2.2 step 3: h_i(sum_{u in S_i(v)} l_i(x_u)) for the
 *                                 sets that can reach v / are reachable from v / neither
 *   policy head ................. Appendix A.7: two-layer feed-forward net, softmax output
 *
 * Readings where the paper is silent (kept identical in the CUDA library):
 *   - what a node sends is f([h_u || x_u]): the raw features are re-injected by
 *     concatenation, otherwise a root would carry no information of its own;
 *   - one progressive sweep in topological order; oracle_embed_sync() is the
 *     paper's literal "repeat the update k times" form and reaches the same
 *     values once k exceeds the depth;
 *   - an empty neighbour set sums to the zero vector;
 *   - the two directions are independent and both start from the raw features;
 *     the node embedding is [h_down || h_up || x];
 *   - S_parents / S_children are strict ancestors / descendants, S_parallel is
 *     the rest without v itself; v enters through the concatenation;
 *   - neighbours are sets: repeated edges count once.
 * Sums run over ascending node id.
 *
 * Layouts: X[n][B][F], H[n][B][d], logits/probs[B][m]; weights W[in][out]
 * row-major, given in float and widened.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef ORACLE_REAL
#define ORACLE_REAL double
#endif
typedef ORACLE_REAL real;

typedef struct {
    int32_t n_layers;           /* 1 or 2 */
    int32_t in_dim, hidden_dim, out_dim;
    const float *W1, *b1, *W2, *b2;
    int32_t act;                /* 0 relu, 1 identity */
    int32_t final_act;          /* 1: activation also after the last layer */
} oracle_mlp;

int oracle_real_bytes(void) { return (int)sizeof(real); }

static real activate(real v, int act) { return (act == 0 && v < 0) ? (real)0 : v; }

/* y = W^T v + b for one layer, W[in][out]. */
static void layer(const float *W, const float *b, int in, int out, const real *v, real *y) {
    for (int j = 0; j < out; ++j) {
        real s = (real)b[j];
        for (int k = 0; k < in; ++k) s += (real)W[(size_t)k * out + j] * v[k];
        y[j] = s;
    }
}

/* Feed-forward net of one or two layers (Appendix A.7). y has out_dim entries. */
static void mlp(const oracle_mlp *M, const real *v, real *y) {
    if (M->n_layers == 1) {
        layer(M->W1, M->b1, M->in_dim, M->out_dim, v, y);
        if (M->final_act) for (int j = 0; j < M->out_dim; ++j) y[j] = activate(y[j], M->act);
        return;
    }
    real *t = (real *)malloc(sizeof(real) * (size_t)M->hidden_dim);
    layer(M->W1, M->b1, M->in_dim, M->hidden_dim, v, t);
    for (int j = 0; j < M->hidden_dim; ++j) t[j] = activate(t[j], M->act);
    layer(M->W2, M->b2, M->hidden_dim, M->out_dim, t, y);
    if (M->final_act) for (int j = 0; j < M->out_dim; ++j) y[j] = activate(y[j], M->act);
    free(t);
}

/* ---- graph helpers ------------------------------------------------------ */

typedef struct {
    int n;
    int *par_ptr, *par;   /* parents of v: par[par_ptr[v] .. par_ptr[v+1]), ascending */
    int *chi_ptr, *chi;   /* children likewise */
    int *topo;            /* a topological order */
} dag;

static int cmp_int(const void *a, const void *b) {
    int x = *(const int *)a, y = *(const int *)b;
    return (x > y) - (x < y);
}

static void dag_free(dag *g) {
    free(g->par_ptr); free(g->par); free(g->chi_ptr); free(g->chi); free(g->topo);
}

/* Builds neighbour sets from an edge list (u -> v). Returns 0, or -1 for an id
 * out of range or a self-loop, -2 for a cycle. */
static int dag_build(dag *g, int n, int64_t n_edges, const int32_t *src, const int32_t *dst) {
    memset(g, 0, sizeof(*g));
    g->n = n;
    for (int64_t e = 0; e < n_edges; ++e)
        if (src[e] < 0 || src[e] >= n || dst[e] < 0 || dst[e] >= n || src[e] == dst[e]) return -1;
    g->par_ptr = (int *)calloc((size_t)n + 1, sizeof(int));
    g->chi_ptr = (int *)calloc((size_t)n + 1, sizeof(int));
    g->par = (int *)malloc(sizeof(int) * (size_t)(n_edges + 1));
    g->chi = (int *)malloc(sizeof(int) * (size_t)(n_edges + 1));
    g->topo = (int *)malloc(sizeof(int) * (size_t)(n + 1));
    /* parents: bucket by dst, sort, drop repeats */
    int *cnt = (int *)calloc((size_t)n + 1, sizeof(int));
    int *tmp = (int *)malloc(sizeof(int) * (size_t)(n_edges + 1));
    for (int pass = 0; pass < 2; ++pass) {
        const int32_t *key = pass == 0 ? dst : src, *val = pass == 0 ? src : dst;
        int *ptr = pass == 0 ? g->par_ptr : g->chi_ptr, *out = pass == 0 ? g->par : g->chi;
        memset(cnt, 0, sizeof(int) * ((size_t)n + 1));
        for (int64_t e = 0; e < n_edges; ++e) cnt[key[e] + 1]++;
        for (int v = 0; v < n; ++v) cnt[v + 1] += cnt[v];
        int *fill = (int *)malloc(sizeof(int) * ((size_t)n + 1));
        memcpy(fill, cnt, sizeof(int) * ((size_t)n + 1));
        for (int64_t e = 0; e < n_edges; ++e) tmp[fill[key[e]]++] = val[e];
        free(fill);
        int w = 0;
        ptr[0] = 0;
        for (int v = 0; v < n; ++v) {
            int a = cnt[v], b = cnt[v + 1];
            qsort(tmp + a, (size_t)(b - a), sizeof(int), cmp_int);
            for (int i = a; i < b; ++i)
                if (i == a || tmp[i] != tmp[i - 1]) out[w++] = tmp[i];
            ptr[v + 1] = w;
        }
    }
    free(cnt); free(tmp);
    /* topological order: repeatedly take nodes whose parents are all taken */
    int *indeg = (int *)malloc(sizeof(int) * ((size_t)n + 1));
    int head = 0, tail = 0;
    for (int v = 0; v < n; ++v) {
        indeg[v] = g->par_ptr[v + 1] - g->par_ptr[v];
        if (indeg[v] == 0) g->topo[tail++] = v;
    }
    while (head < tail) {
        int u = g->topo[head++];
        for (int i = g->chi_ptr[u]; i < g->chi_ptr[u + 1]; ++i)
            if (--indeg[g->chi[i]] == 0) g->topo[tail++] = g->chi[i];
    }
    free(indeg);
    if (tail != n) { dag_free(g); return -2; }
    return 0;
}

/* ---- step 1: raw features (Sec. 2.1; Sec. 2.2 step 1) -------------------- */

/* x = [cost, bytes, one-hot(device, m), is-current, is-placed]; F = m + 4. */
int oracle_features(int32_t n, int32_t B, int32_t m, const float *cost, const float *bytes,
                    const uint8_t *dev /*[B][n]*/, const int32_t *cur /*[B]*/,
                    const uint8_t *placed /*[B][n]*/, real *X /*[n][B][m+4]*/) {
    const int F = m + 4;
    for (int v = 0; v < n; ++v)
        for (int b = 0; b < B; ++b) {
            real *x = X + ((size_t)v * B + b) * F;
            x[0] = (real)cost[v];
            x[1] = (real)bytes[v];
            for (int k = 0; k < m; ++k) x[2 + k] = (dev[(size_t)b * n + v] == k) ? 1 : 0;
            x[2 + m] = (cur[b] == v) ? 1 : 0;
            x[3 + m] = placed[(size_t)b * n + v] ? 1 : 0;
        }
    return 0;
}

/* ---- step 2: two-way message passing (Sec. 2.2 step 2) ------------------- */

/* h_v = g( sum_{u in nbr(v)} f([h_u || x_u]) ) for one state and one direction.
 * order: nodes such that every neighbour of v precedes v. */
static void sweep(const dag *g, int down, const int *order, int B, int b, int F, int d,
                  const real *X, const oracle_mlp *f, const oracle_mlp *gg, real *H) {
    const int n = g->n;
    real *s = (real *)malloc(sizeof(real) * (size_t)d);
    real *msg = (real *)malloc(sizeof(real) * (size_t)d);
    real *in = (real *)malloc(sizeof(real) * (size_t)(d + F));
    for (int i = 0; i < n; ++i) {
        int v = order[i];
        const int *ptr = down ? g->par_ptr : g->chi_ptr, *nbr = down ? g->par : g->chi;
        for (int j = 0; j < d; ++j) s[j] = 0;
        for (int e = ptr[v]; e < ptr[v + 1]; ++e) {
            int u = nbr[e];
            memcpy(in, H + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);
            memcpy(in + d, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);
            mlp(f, in, msg);
            for (int j = 0; j < d; ++j) s[j] += msg[j];
        }
        mlp(gg, s, H + ((size_t)v * B + b) * d);
    }
    free(s); free(msg); free(in);
}

int oracle_embed(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                 int32_t B, int32_t F, int32_t d, const real *X /*[n][B][F]*/,
                 const oracle_mlp *f_down, const oracle_mlp *g_down,
                 const oracle_mlp *f_up, const oracle_mlp *g_up,
                 real *H_down /*[n][B][d]*/, real *H_up /*[n][B][d]*/, int32_t n_threads) {
    dag g;
    int rc = dag_build(&g, n, n_edges, src, dst);
    if (rc) return rc;
    int *rev = (int *)malloc(sizeof(int) * ((size_t)n + 1));
    for (int i = 0; i < n; ++i) rev[i] = g.topo[n - 1 - i];
    (void)n_threads;
#pragma omp parallel for schedule(dynamic) num_threads(n_threads > 0 ? n_threads : 1)
    for (int b = 0; b < B; ++b) {
        sweep(&g, 1, g.topo, B, b, F, d, X, f_down, g_down, H_down);
        sweep(&g, 0, rev, B, b, F, d, X, f_up, g_up, H_up);
    }
    free(rev);
    dag_free(&g);
    return 0;
}

/* The synchronous form of the same update (Sec. 2.2 step 2, "repeat the
 * message passing updates k times"): all nodes are updated at once from the
 * previous round's values, starting from zeros, for `rounds` rounds. */
int oracle_embed_sync(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                      int32_t B, int32_t F, int32_t d, const real *X,
                      const oracle_mlp *f_down, const oracle_mlp *g_down,
                      const oracle_mlp *f_up, const oracle_mlp *g_up,
                      int32_t rounds, real *H_down, real *H_up) {
    dag g;
    int rc = dag_build(&g, n, n_edges, src, dst);
    if (rc) return rc;
    size_t tot = (size_t)n * B * d;
    real *prev = (real *)malloc(sizeof(real) * (tot + 1));
    real *s = (real *)malloc(sizeof(real) * (size_t)d);
    real *msg = (real *)malloc(sizeof(real) * (size_t)d);
    real *in = (real *)malloc(sizeof(real) * (size_t)(d + F));
    for (int dir = 0; dir < 2; ++dir) {
        real *H = dir == 0 ? H_down : H_up;
        const oracle_mlp *f = dir == 0 ? f_down : f_up, *gg = dir == 0 ? g_down : g_up;
        const int *ptr = dir == 0 ? g.par_ptr : g.chi_ptr, *nbr = dir == 0 ? g.par : g.chi;
        for (size_t i = 0; i < tot; ++i) H[i] = 0;
        for (int r = 0; r < rounds; ++r) {
            memcpy(prev, H, sizeof(real) * tot);
            for (int v = 0; v < n; ++v)
                for (int b = 0; b < B; ++b) {
                    for (int j = 0; j < d; ++j) s[j] = 0;
                    for (int e = ptr[v]; e < ptr[v + 1]; ++e) {
                        int u = nbr[e];
                        memcpy(in, prev + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);
                        memcpy(in + d, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);
                        mlp(f, in, msg);
                        for (int j = 0; j < d; ++j) s[j] += msg[j];
                    }
                    mlp(gg, s, H + ((size_t)v * B + b) * d);
                }
        }
    }
    free(prev); free(s); free(msg); free(in);
    dag_free(&g);
    return 0;
}

/* ---- step 3 + head: group pooling, policy head, softmax ------------------ */

/* Marks every node reachable from c along `ptr/nbr` (c itself excluded). */
static void reach(int n, const int *ptr, const int *nbr, int c, uint8_t *mark, int *stack) {
    memset(mark, 0, (size_t)n);
    int top = 0;
    stack[top++] = c;
    while (top) {
        int u = stack[--top];
        for (int e = ptr[u]; e < ptr[u + 1]; ++e) {
            int w = nbr[e];
            if (!mark[w]) { mark[w] = 1; stack[top++] = w; }
        }
    }
}

int oracle_policy(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                  int32_t B, int32_t F, int32_t d, int32_t m,
                  const real *X, const real *H_down, const real *H_up, const int32_t *cur,
                  const oracle_mlp *l /*[3]: parents, children, parallel*/,
                  const oracle_mlp *h /*[3]*/, const oracle_mlp *head,
                  real *logits /*[B][m]*/, real *probs /*[B][m]*/, int32_t n_threads) {
    dag g;
    int rc = dag_build(&g, n, n_edges, src, dst);
    if (rc) return rc;
    for (int b = 0; b < B; ++b) if (cur[b] < 0 || cur[b] >= n) { dag_free(&g); return -3; }
    const int E = 2 * d + F, Z = 5 * d + F;
    (void)n_threads;
#pragma omp parallel for schedule(dynamic) num_threads(n_threads > 0 ? n_threads : 1)
    for (int b = 0; b < B; ++b) {
        uint8_t *anc = (uint8_t *)malloc((size_t)n + 1), *desc = (uint8_t *)malloc((size_t)n + 1);
        int *stack = (int *)malloc(sizeof(int) * ((size_t)n + 1));
        real *e = (real *)malloc(sizeof(real) * (size_t)E);
        real *y = (real *)malloc(sizeof(real) * (size_t)d);
        real *sum = (real *)malloc(sizeof(real) * (size_t)(3 * d));
        real *z = (real *)malloc(sizeof(real) * (size_t)Z);
        const int c = cur[b];
        reach(n, g.par_ptr, g.par, c, anc, stack);    /* nodes that can reach c */
        reach(n, g.chi_ptr, g.chi, c, desc, stack);   /* nodes reachable from c */
        for (int j = 0; j < 3 * d; ++j) sum[j] = 0;
        for (int u = 0; u < n; ++u) {
            memcpy(e, H_down + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);
            memcpy(e + d, H_up + ((size_t)u * B + b) * d, sizeof(real) * (size_t)d);
            memcpy(e + 2 * d, X + ((size_t)u * B + b) * F, sizeof(real) * (size_t)F);
            if (u == c) { memcpy(z, e, sizeof(real) * (size_t)E); continue; }
            int i = anc[u] ? 0 : (desc[u] ? 1 : 2);
            mlp(&l[i], e, y);
            for (int j = 0; j < d; ++j) sum[i * d + j] += y[j];
        }
        for (int i = 0; i < 3; ++i) mlp(&h[i], sum + i * d, z + E + i * d);
        real *lg = logits + (size_t)b * m;
        mlp(head, z, lg);
        if (probs) {
            real mx = lg[0], tot = 0;
            for (int k = 1; k < m; ++k) if (lg[k] > mx) mx = lg[k];
            for (int k = 0; k < m; ++k) { probs[(size_t)b * m + k] = (real)exp((double)(lg[k] - mx)); tot += probs[(size_t)b * m + k]; }
            for (int k = 0; k < m; ++k) probs[(size_t)b * m + k] /= tot;
        }
        free(anc); free(desc); free(stack); free(e); free(y); free(sum); free(z);
    }
    dag_free(&g);
    return 0;
}

/* Sizes of the three sets for node c (for partition checks). */
int oracle_group_sizes(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                       int32_t c, int32_t *sizes /*[3]*/, uint8_t *group /*[n]: 0 anc,1 desc,2 parallel,3 self*/) {
    dag g;
    int rc = dag_build(&g, n, n_edges, src, dst);
    if (rc) return rc;
    uint8_t *anc = (uint8_t *)malloc((size_t)n + 1), *desc = (uint8_t *)malloc((size_t)n + 1);
    int *stack = (int *)malloc(sizeof(int) * ((size_t)n + 1));
    reach(n, g.par_ptr, g.par, c, anc, stack);
    reach(n, g.chi_ptr, g.chi, c, desc, stack);
    sizes[0] = sizes[1] = sizes[2] = 0;
    for (int u = 0; u < n; ++u) {
        int i = (u == c) ? 3 : (anc[u] ? 0 : (desc[u] ? 1 : 2));
        if (i < 3) sizes[i]++;
        if (group) group[u] = (uint8_t)i;
    }
    free(anc); free(desc); free(stack);
    dag_free(&g);
    return 0;
}
