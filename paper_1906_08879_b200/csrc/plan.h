// Host-side plan of a DAG: level schedule of the message passing (Sec. 2.2
// step 2 of the Placeto paper) and the pairwise reachability relation that
// defines the three pooling sets (Sec. 2.2 step 3). Pure C++, no CUDA.
#pragma once
#include <cstdint>
#include <vector>

#include "placeto.h"

namespace placeto {

struct LevelPlan {
    int32_t n_levels = 0;
    std::vector<int32_t> level_ptr;  // [n_levels + 1] positions into order
    std::vector<int32_t> order;      // [n] node ids by level, ascending id inside a level
    std::vector<int32_t> nbr_ptr;    // [n + 1] by position in order
    std::vector<int32_t> nbr;        // neighbour ids (parents for down, children for up)
    // On-chip message slots. A node's message f([h || x]) is live from its own
    // level until the last level that consumes it; nodes whose lifetimes do not
    // overlap share a slot, so a block can keep all live messages of its states
    // in shared memory instead of n rows in global memory.
    int32_t n_slots = 0;
    std::vector<int32_t> own_slot;   // [n] by position: slot the node writes, -1 if nobody reads it
    std::vector<int32_t> nbr_slot;   // [nbr.size()] slot of each neighbour
};

struct HostPlan {
    int32_t n = 0;
    int64_t n_edges = 0;             // distinct edges
    int32_t max_level_width = 0;     // over both directions
    int32_t max_degree = 0;          // largest neighbour set, both directions
    LevelPlan dir[2];                // 0 top-down, 1 bottom-up
    std::vector<uint8_t> relation;   // [n * n], see placeto_graph_host_view
    // by node id, for the runtime simulator: children (ascending) and number of parents
    std::vector<int32_t> child_ptr, child, n_parents;
    std::vector<int32_t> parent_ptr, parent;   // by node id, ascending (the policy gradient's gathers)
};

// Validates the edge list and fills `plan`. Returns PLACETO_OK,
// PLACETO_ERR_INVALID_ARG, PLACETO_ERR_NOT_DAG or PLACETO_ERR_NO_MEMORY.
placeto_status build_plan(int32_t n, int64_t n_edges, const int32_t *src, const int32_t *dst,
                          HostPlan &plan);

}  // namespace placeto
