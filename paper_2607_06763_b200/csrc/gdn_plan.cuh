// The tree-plan computation for one tree (Section 3.4.2, "computed once per decode step"): depth and root-path list of
// every node, and for trees of more than 64 nodes the depth-first numbering cut into ancestor-closed groups, with one
// record per group appended to the unit list that the tensor-core verify kernel walks (see gdn_internal.cuh for the
// layouts).  A device function, so that it can run as a kernel of its own (gdn_plan.cu) or as extra CTAs in front of
// the commit kernel's (gdn_commit.cu: the fused call on trees of more than 64 nodes).  One CTA of PLAN_THREADS
// threads per tree.
#pragma once

#include "gdn_internal.cuh"

namespace gdn {

constexpr int PLAN_THREADS = 256;

struct PlanArgs {
    int n_seq, total_nodes, max_tree_nodes, max_depth;
    const int32_t *parent, *node_offsets, *n_nodes;   // node_offsets == nullptr: padded layout, node counts in n_nodes
    int32_t *tree_ok;
    uint8_t *depth;
    uint16_t *anc;
    uint8_t *anc8;
    uint16_t *dfs_node;
    uint8_t *dfs_depth, *dfs_anc8;
    uint16_t *group_start;
    int32_t *unit_count;
    uint4 *unit_list;
    int32_t *status_dev;
};

inline PlanArgs plan_args(const gdn_shape_t &s, const int32_t *parent, const int32_t *node_offsets,
                          const int32_t *n_nodes, const PlanPtrs &plan, int32_t *status_dev)
{
    return {s.n_seq, s.total_nodes, s.max_tree_nodes, s.max_depth, parent, node_offsets, n_nodes, plan.tree_ok,
            plan.depth, plan.anc, plan.anc8, plan.dfs_node, plan.dfs_depth, plan.dfs_anc8, plan.group_start,
            plan.unit_count, plan.unit_list, status_dev};
}

#ifdef __CUDACC__
__device__ __forceinline__ void plan_tree(const PlanArgs &a, const int b)
{
    const int n_seq = a.n_seq, total_nodes = a.total_nodes, max_tree_nodes = a.max_tree_nodes, max_depth = a.max_depth;
    const int32_t *__restrict__ parent = a.parent;
    const int32_t *__restrict__ node_offsets = a.node_offsets;
    const int32_t *__restrict__ n_nodes = a.n_nodes;
    int32_t *__restrict__ tree_ok = a.tree_ok;
    uint8_t *__restrict__ depth = a.depth;
    uint16_t *__restrict__ anc = a.anc;
    uint8_t *__restrict__ anc8 = a.anc8;
    uint16_t *dfs_node = a.dfs_node;
    uint8_t *__restrict__ dfs_depth = a.dfs_depth;
    uint8_t *__restrict__ dfs_anc8 = a.dfs_anc8;
    uint16_t *__restrict__ group_start = a.group_start;
    int32_t *unit_count = a.unit_count;
    uint4 *__restrict__ unit_list = a.unit_list;
    int32_t *status_dev = a.status_dev;

    __shared__ int size_s[GDN_GROUPED_MAX_NODES];        // subtree sizes
    __shared__ uint16_t left_s[GDN_GROUPED_MAX_NODES];   // nodes in the subtrees of earlier siblings
    __shared__ uint16_t pos_s[GDN_GROUPED_MAX_NODES];    // pre-order position of node i
    __shared__ uint8_t depth_at_s[GDN_GROUPED_MAX_NODES];   // depth of the node at pre-order position r
    __shared__ uint16_t gstart_s[GDN_MAX_GROUPS + 1];        // first position of each group (then the tree's size)
    // parent[] of this tree, staged once so that the root-path walks below run out of shared memory
    __shared__ int32_t par_s[GDN_MAX_TREE_NODES];
    if (b == 0 && threadIdx.x == 0) unit_count[1] = plan_magic(n_seq, max_tree_nodes, max_depth);
    // ragged packing: the tree's rows by node_offsets[]; padded layout: max_tree_nodes rows per tree, n_nodes[b] used
    const int lo = node_offsets ? node_offsets[b] : b * max_tree_nodes;
    const int hi = node_offsets ? node_offsets[b + 1] : lo + n_nodes[b];
    const int T = hi - lo;
    bool offsets_ok = lo >= 0 && T >= 0 && T <= max_tree_nodes && hi <= total_nodes;
    if (node_offsets && b == 0) offsets_ok = offsets_ok && lo == 0;
    if (node_offsets && b == n_seq - 1) offsets_ok = offsets_ok && hi == total_nodes;
    if (!offsets_ok) {
        if (threadIdx.x == 0) {
            report_status(status_dev, GDN_ERR_TREE);
            tree_ok[b] = 0;
            if (n_seq == 1) *unit_count = 0;
        }
        return;   // no record in the unit list: nothing of this tree is verified
    }
    const bool grouped = max_depth <= 16 && T > 64 && T <= GDN_GROUPED_MAX_NODES;
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        par_s[i] = parent[lo + i];
        if (grouped) size_s[i] = 1;
    }
    __syncthreads();
    int err = 0;
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        // first walk: count the nodes on the root path, checking parent[] as we go
        int d = 0, cur = i;
        while (cur >= 0) {
            if (++d > max_depth) { err = GDN_ERR_DEPTH; break; }
            const int p = par_s[cur];
            if (p < -1 || p >= cur) { err = GDN_ERR_TREE; break; }
            cur = p;
        }
        if (err) break;
        depth[lo + i] = (uint8_t)d;
        // second walk: fill the list root first, the node itself last
        uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        cur = i;
        uint32_t w0 = 0xFFFFFFFFu, w1 = 0xFFFFFFFFu, w2 = 0xFFFFFFFFu, w3 = 0xFFFFFFFFu;
        for (int t = d - 1; t >= 0; --t) {
            row[t] = (uint16_t)cur;
            // the same list as bytes, one 16-byte row per node (used when max_depth <= 16, T <= 256)
            const uint32_t keep = ~(0xFFu << ((t & 3) * 8)), put = ((uint32_t)cur & 0xFFu) << ((t & 3) * 8);
            if ((t >> 2) == 0) w0 = (w0 & keep) | put;
            else if ((t >> 2) == 1) w1 = (w1 & keep) | put;
            else if ((t >> 2) == 2) w2 = (w2 & keep) | put;
            else if ((t >> 2) == 3) w3 = (w3 & keep) | put;
            cur = par_s[cur];
            if (grouped && cur >= 0) atomicAdd(&size_s[cur], 1);   // node i lies in the subtree of each proper ancestor
        }
        if (max_depth <= 16 && T <= 256)
            *reinterpret_cast<uint4 *>(anc8 + (size_t)(lo + i) * 16) = make_uint4(w0, w1, w2, w3);
    }
    const int any_err = __syncthreads_or(err != 0);
    if (err) report_status(status_dev, err);
    if (threadIdx.x == 0) tree_ok[b] = any_err ? 0 : 1;
    if (any_err || !grouped) {
        // a tree that fits one tile is its own single group with the identity numbering, marked by n_prefix =
        // 0xFFFF (no group at all if the tree was rejected or is empty)
        // (a call with a single tree keeps the count itself; otherwise the counter was zeroed in front of this grid)
        const bool one = !any_err && T > 0 && T <= GDN_GROUP_TILE;
        if (threadIdx.x == 0 && n_seq == 1) *unit_count = one ? 1 : 0;
        if (threadIdx.x == 0 && one)
            unit_list[n_seq == 1 ? 0 : atomicAdd(unit_count, 1)] =
                make_uint4((uint32_t)b, (uint32_t)lo, (uint32_t)T << 16, 0xFFFFu);
        return;
    }

    // Pre-order position = (#proper ancestors) + sum over the root path of the sizes of the subtrees
    // hanging off earlier siblings (roots count as siblings of one another; siblings by increasing id).
    // With a breadth-first numbering (parent[] non-decreasing, what tree builders emit) the siblings of a node are
    // its neighbours: the earlier ones are the run in front of it; any other topological numbering is searched.
    bool sorted_here = true;
    for (int i = threadIdx.x + 1; i < T; i += PLAN_THREADS) sorted_here = sorted_here && par_s[i] >= par_s[i - 1];
    const bool sorted = __syncthreads_and(sorted_here);
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const int p = par_s[i];
        int acc = 0;
        if (sorted) {
            for (int j = i - 1; j > p && par_s[j] == p; --j) acc += size_s[j];
        } else {
            for (int j = p + 1; j < i; ++j)
                if (par_s[j] == p) acc += size_s[j];
        }
        left_s[i] = (uint16_t)acc;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        const int d = depth[lo + i];
        int pos = d - 1;
        for (int t = 0; t < d; ++t) pos += left_s[row[t]];
        pos_s[i] = (uint16_t)pos;
        dfs_node[lo + pos] = (uint16_t)i;
        dfs_depth[lo + pos] = (uint8_t)d;
        depth_at_s[pos] = (uint8_t)d;
    }
    __syncthreads();
    // Groups: each takes as many positions as the tile leaves after the proper ancestors of its first node
    if (threadIdx.x == 0) {
        int start = 0, k = 0;
        while (start < T && k < GDN_MAX_GROUPS) {
            gstart_s[k++] = (uint16_t)start;
            start += GDN_GROUP_TILE - (depth_at_s[start] - 1);
        }
        for (; k <= GDN_MAX_GROUPS; ++k) gstart_s[k] = (uint16_t)T;
    }
    __syncthreads();
    for (int k = threadIdx.x; k <= GDN_MAX_GROUPS; k += PLAN_THREADS)
        group_start[(size_t)b * (GDN_MAX_GROUPS + 1) + k] = gstart_s[k];
    // one record per group in the unit list, the groups of this tree next to one another
    __shared__ int list_base_s;
    if (threadIdx.x == 0) {
        int n_groups = 0;
        while (n_groups < GDN_MAX_GROUPS && gstart_s[n_groups] < T) ++n_groups;
        if (n_seq == 1) {
            *unit_count = n_groups;
            list_base_s = 0;
        } else {
            list_base_s = atomicAdd(unit_count, n_groups);
        }
    }
    __syncthreads();
    for (int k = threadIdx.x; k < GDN_MAX_GROUPS; k += PLAN_THREADS) {
        const int g0 = gstart_s[k], own = gstart_s[k + 1] - g0;
        if (own > 0)   // (first position, own nodes), (n_prefix, node at the first position)
            unit_list[list_base_s + k] = make_uint4((uint32_t)b, (uint32_t)lo, (uint32_t)g0 | ((uint32_t)own << 16),
                                                    (uint32_t)(depth_at_s[g0] - 1) | ((uint32_t)dfs_node[lo + g0] << 16));
    }
    // Root path of every node in the virtual indices of its group: an ancestor before the group's first
    // position is an ancestor of the group's first node and gets index depth-1; one inside the group gets
    // n_prefix + its offset in the group, n_prefix = depth(first node) - 1.
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        const int d = depth[lo + i];
        const int pos = pos_s[i];
        int k = 0;
        while (gstart_s[k + 1] <= pos) ++k;   // the group of this position (at most GDN_MAX_GROUPS steps)
        const int g0 = gstart_s[k];
        const int n_prefix = depth_at_s[g0] - 1;
        uint32_t w[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
        for (int t = 0; t < d; ++t) {
            const int pa = pos_s[row[t]];
            const uint32_t v = pa < g0 ? (uint32_t)t : (uint32_t)(n_prefix + pa - g0);
            w[t >> 2] = (w[t >> 2] & ~(0xFFu << ((t & 3) * 8))) | (v << ((t & 3) * 8));
        }
        *reinterpret_cast<uint4 *>(dfs_anc8 + (size_t)(lo + pos) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}
#endif

}  // namespace gdn
