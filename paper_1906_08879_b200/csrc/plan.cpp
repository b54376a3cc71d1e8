// Host graph builder: validation, level bucketing, CSR in level order and the
// reachability relation. See plan.h.
#include "plan.h"

#include <algorithm>
#include <new>

namespace placeto {

namespace {

// Longest-path layering along one direction. `nbrs[v]` are the nodes v waits
// for (parents for the top-down pass), `rev[v]` the nodes waiting for v.
// Returns false if the graph has a cycle.
bool layer(int32_t n, const std::vector<std::vector<int32_t>> &nbrs,
           const std::vector<std::vector<int32_t>> &rev, std::vector<int32_t> &level) {
    std::vector<int32_t> pending(n);
    std::vector<int32_t> queue;
    queue.reserve(n);
    level.assign(n, 0);
    for (int32_t v = 0; v < n; ++v) {
        pending[v] = static_cast<int32_t>(nbrs[v].size());
        if (pending[v] == 0) queue.push_back(v);
    }
    for (size_t head = 0; head < queue.size(); ++head) {
        const int32_t u = queue[head];
        for (int32_t v : rev[u]) {
            level[v] = std::max(level[v], level[u] + 1);
            if (--pending[v] == 0) queue.push_back(v);
        }
    }
    return static_cast<int32_t>(queue.size()) == n;
}

void bucket(int32_t n, const std::vector<int32_t> &level,
            const std::vector<std::vector<int32_t>> &nbrs, LevelPlan &out) {
    int32_t n_levels = 0;
    for (int32_t v = 0; v < n; ++v) n_levels = std::max(n_levels, level[v] + 1);
    out.n_levels = n_levels;
    out.level_ptr.assign(n_levels + 1, 0);
    for (int32_t v = 0; v < n; ++v) out.level_ptr[level[v] + 1]++;
    for (int32_t l = 0; l < n_levels; ++l) out.level_ptr[l + 1] += out.level_ptr[l];
    out.order.assign(n, 0);
    std::vector<int32_t> fill(out.level_ptr.begin(), out.level_ptr.end() - 1);
    for (int32_t v = 0; v < n; ++v) out.order[fill[level[v]]++] = v;  // ascending id per level
    out.nbr_ptr.assign(n + 1, 0);
    out.nbr.clear();
    for (int32_t p = 0; p < n; ++p) {
        const auto &list = nbrs[out.order[p]];
        out.nbr.insert(out.nbr.end(), list.begin(), list.end());
        out.nbr_ptr[p + 1] = static_cast<int32_t>(out.nbr.size());
    }
}

// Greedy slot assignment in level order. A slot freed by a node whose last
// consumer sits in level l can be taken again from level l + 1 on (all rows of
// a level may run concurrently, so a slot is never reused inside the level that
// still reads it).
void assign_slots(int32_t n, const std::vector<int32_t> &level, LevelPlan &out) {
    std::vector<int32_t> last_use(n, -1);
    for (int32_t p = 0; p < n; ++p)
        for (int32_t e = out.nbr_ptr[p]; e < out.nbr_ptr[p + 1]; ++e)
            last_use[out.nbr[e]] = std::max(last_use[out.nbr[e]], level[out.order[p]]);
    std::vector<std::vector<int32_t>> release(out.n_levels + 1);   // slots free from this level on
    std::vector<int32_t> free_slots, slot_of(n, -1);
    int32_t n_slots = 0;
    out.own_slot.assign(n, -1);
    for (int32_t l = 0; l < out.n_levels; ++l) {
        for (int32_t s : release[l]) free_slots.push_back(s);
        for (int32_t p = out.level_ptr[l]; p < out.level_ptr[l + 1]; ++p) {
            const int32_t v = out.order[p];
            if (last_use[v] < 0) continue;
            int32_t s;
            if (!free_slots.empty()) { s = free_slots.back(); free_slots.pop_back(); }
            else s = n_slots++;
            slot_of[v] = s;
            out.own_slot[p] = s;
            release[last_use[v] + 1].push_back(s);
        }
    }
    out.n_slots = n_slots;
    out.nbr_slot.resize(out.nbr.size());
    for (size_t e = 0; e < out.nbr.size(); ++e) out.nbr_slot[e] = slot_of[out.nbr[e]];
}

}  // namespace

placeto_status build_plan(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                          HostPlan &plan) {
    if (n < 1 || n > PLACETO_MAX_NODES || n_edges < 0) return PLACETO_ERR_INVALID_ARG;
    if (n_edges > 0 && (src == nullptr || dst == nullptr)) return PLACETO_ERR_INVALID_ARG;
    try {
        std::vector<std::vector<int32_t>> par(n), chi(n);
        for (int64_t e = 0; e < n_edges; ++e) {
            const int32_t u = src[e], v = dst[e];
            if (u < 0 || u >= n || v < 0 || v >= n || u == v) return PLACETO_ERR_NOT_DAG;
            par[v].push_back(u);
            chi[u].push_back(v);
        }
        int64_t distinct = 0;
        int32_t max_degree = 0;
        for (int32_t v = 0; v < n; ++v) {
            for (auto *list : {&par[v], &chi[v]}) {
                std::sort(list->begin(), list->end());
                list->erase(std::unique(list->begin(), list->end()), list->end());
                max_degree = std::max(max_degree, static_cast<int32_t>(list->size()));
            }
            distinct += static_cast<int64_t>(par[v].size());
        }
        std::vector<int32_t> level_down, level_up;
        if (!layer(n, par, chi, level_down)) return PLACETO_ERR_NOT_DAG;
        if (!layer(n, chi, par, level_up)) return PLACETO_ERR_NOT_DAG;
        plan.n = n;
        plan.n_edges = distinct;
        plan.max_degree = max_degree;
        bucket(n, level_down, par, plan.dir[0]);
        bucket(n, level_up, chi, plan.dir[1]);
        assign_slots(n, level_down, plan.dir[0]);
        assign_slots(n, level_up, plan.dir[1]);
        plan.child_ptr.assign(n + 1, 0);
        plan.child.clear();
        plan.n_parents.assign(n, 0);
        for (int32_t v = 0; v < n; ++v) {
            plan.child.insert(plan.child.end(), chi[v].begin(), chi[v].end());
            plan.child_ptr[v + 1] = static_cast<int32_t>(plan.child.size());
            plan.n_parents[v] = static_cast<int32_t>(par[v].size());
        }
        plan.parent_ptr.assign(n + 1, 0);
        plan.parent.clear();
        for (int32_t v = 0; v < n; ++v) {
            plan.parent.insert(plan.parent.end(), par[v].begin(), par[v].end());
            plan.parent_ptr[v + 1] = static_cast<int32_t>(plan.parent.size());
        }
        plan.max_level_width = 0;
        for (int dir = 0; dir < 2; ++dir)
            for (int32_t l = 0; l < plan.dir[dir].n_levels; ++l)
                plan.max_level_width = std::max(
                    plan.max_level_width, plan.dir[dir].level_ptr[l + 1] - plan.dir[dir].level_ptr[l]);

        // Ancestor bitsets in top-down level order: anc(v) = U_{u in par(v)} (anc(u) + u).
        const size_t words = (static_cast<size_t>(n) + 63) / 64;
        std::vector<uint64_t> anc(static_cast<size_t>(n) * words, 0);
        for (int32_t p = 0; p < n; ++p) {
            const int32_t v = plan.dir[0].order[p];
            uint64_t *av = &anc[static_cast<size_t>(v) * words];
            for (int32_t u : par[v]) {
                const uint64_t *au = &anc[static_cast<size_t>(u) * words];
                for (size_t w = 0; w < words; ++w) av[w] |= au[w];
                av[u >> 6] |= 1ull << (u & 63);
            }
        }
        plan.relation.assign(static_cast<size_t>(n) * n, 2);
        for (int32_t c = 0; c < n; ++c) {
            const uint64_t *ac = &anc[static_cast<size_t>(c) * words];
            uint8_t *row = &plan.relation[static_cast<size_t>(c) * n];
            for (int32_t u = 0; u < n; ++u)
                if (ac[u >> 6] >> (u & 63) & 1) {
                    row[u] = 0;                                         // u can reach c
                    plan.relation[static_cast<size_t>(u) * n + c] = 1;  // u can reach c, seen from u
                }
            row[c] = 3;
        }
    } catch (const std::bad_alloc &) {
        return PLACETO_ERR_NO_MEMORY;
    }
    return PLACETO_OK;
}

}  // namespace placeto
