// Tree metadata ("computed once per decode step", Section 3.4.2): for every node its depth and
// the list of nodes on its root path.  The ancestor sets of Section 3.4.2 are kept as explicit
// root-first lists rather than bitmasks: with at most max_depth (16 in the paper) nodes per path a
// list is smaller than a T-bit mask for T > 256 and lets the solve visit only real ancestors.
// For small trees the kernel also emits a depth-first (pre-order) numbering: in that order the
// ancestors of the current node are exactly the current stack, which is what lets the tensor-core
// verify kernel keep the solve results of a root path in registers.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int PLAN_THREADS = 128;
constexpr int PLAN_DFS_MAX = 256;   // trees up to this size get the depth-first tables

__global__ void __launch_bounds__(PLAN_THREADS)
plan_kernel(int n_seq, int total_nodes, int max_tree_nodes, int max_depth,
            const int32_t *__restrict__ parent, const int32_t *__restrict__ node_offsets,
            int32_t *__restrict__ tree_ok, uint8_t *__restrict__ depth, uint16_t *__restrict__ anc,
            uint8_t *__restrict__ order8, uint8_t *__restrict__ dpos8, uint8_t *__restrict__ ancpos8,
            int32_t *status_dev)
{
    __shared__ int16_t par_s[PLAN_DFS_MAX];
    __shared__ int16_t left_s[PLAN_DFS_MAX];    // nodes before i among the subtrees of its earlier siblings
    __shared__ int size_s[PLAN_DFS_MAX];        // subtree size
    __shared__ uint8_t pos_s[PLAN_DFS_MAX];     // pre-order position

    const int b = blockIdx.x;
    const int lo = node_offsets[b], hi = node_offsets[b + 1];
    const int T = hi - lo;
    bool offsets_ok = lo >= 0 && T >= 0 && T <= max_tree_nodes && hi <= total_nodes;
    if (b == 0) offsets_ok = offsets_ok && lo == 0;
    if (b == n_seq - 1) offsets_ok = offsets_ok && hi == total_nodes;
    if (!offsets_ok) {
        if (threadIdx.x == 0) {
            report_status(status_dev, GDN_ERR_TREE);
            tree_ok[b] = 0;
        }
        return;
    }
    const bool dfs = max_depth <= 16 && T <= PLAN_DFS_MAX;
    if (dfs)
        for (int i = threadIdx.x; i < T; i += PLAN_THREADS) size_s[i] = 1;
    __syncthreads();

    int err = 0;
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        // first walk: count the nodes on the root path, checking parent[] as we go
        int d = 0, cur = i;
        while (cur >= 0) {
            if (++d > max_depth) { err = GDN_ERR_DEPTH; break; }
            const int p = parent[lo + cur];
            if (p < -1 || p >= cur) { err = GDN_ERR_TREE; break; }
            cur = p;
        }
        if (err) break;
        depth[lo + i] = (uint8_t)d;
        // second walk: fill the list root first, the node itself last
        uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        cur = i;
        for (int t = d - 1; t >= 0; --t) {
            row[t] = (uint16_t)cur;
            cur = parent[lo + cur];
            if (dfs && cur >= 0) atomicAdd(&size_s[cur], 1);   // i lies in the subtree of each proper ancestor
        }
        if (dfs) par_s[i] = (int16_t)parent[lo + i];
    }
    const int any_err = __syncthreads_or(err != 0);
    if (err) report_status(status_dev, err);
    if (threadIdx.x == 0) tree_ok[b] = any_err ? 0 : 1;
    if (any_err || !dfs) return;

    // pre-order position = (#proper ancestors) + sum over the root path of the sizes of the
    // subtrees hanging off earlier siblings (roots count as siblings of one another)
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const int p = par_s[i];
        int acc = 0;
        for (int j = (p < 0 ? 0 : p + 1); j < i; ++j)
            if (par_s[j] == p) acc += size_s[j];
        left_s[i] = (int16_t)acc;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        const int d = depth[lo + i];
        int pos = d - 1;
        for (int t = 0; t < d; ++t) pos += left_s[row[t]];
        pos_s[i] = (uint8_t)pos;
        order8[lo + pos] = (uint8_t)i;
        dpos8[lo + pos] = (uint8_t)d;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) {
        const uint16_t *row = anc + (size_t)(lo + i) * max_depth;
        const int d = depth[lo + i];
        uint32_t w[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
        for (int t = 0; t < d; ++t) {
            const uint32_t v = pos_s[row[t]];
            w[t >> 2] = (w[t >> 2] & ~(0xFFu << ((t & 3) * 8))) | (v << ((t & 3) * 8));
        }
        *reinterpret_cast<uint4 *>(ancpos8 + (size_t)(lo + pos_s[i]) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace

cudaError_t launch_plan(const gdn_shape_t &s, const int32_t *parent, const int32_t *node_offsets,
                        const PlanPtrs &plan, int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0) return cudaSuccess;
    plan_kernel<<<s.n_seq, PLAN_THREADS, 0, stream>>>(s.n_seq, s.total_nodes, s.max_tree_nodes,
                                                      s.max_depth, parent, node_offsets, plan.tree_ok,
                                                      plan.depth, plan.anc, plan.order8, plan.dpos8,
                                                      plan.ancpos8, status_dev);
    return cudaGetLastError();
}

}  // namespace gdn
