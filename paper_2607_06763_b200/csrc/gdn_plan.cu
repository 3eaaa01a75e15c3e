// Tree metadata ("computed once per decode step", Section 3.4.2): for every node its depth and
// the list of nodes on its root path.  The ancestor sets of Section 3.4.2 are kept as explicit
// root-first lists rather than bitmasks: with at most max_depth (16 in the paper) nodes per path a
// list is smaller than a T-bit mask for T > 256 and lets the solve visit only real ancestors.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int PLAN_THREADS = 128;

__global__ void __launch_bounds__(PLAN_THREADS)
plan_kernel(int n_seq, int total_nodes, int max_tree_nodes, int max_depth,
            const int32_t *__restrict__ parent, const int32_t *__restrict__ node_offsets,
            int32_t *__restrict__ tree_ok, uint8_t *__restrict__ depth, uint16_t *__restrict__ anc,
            uint8_t *__restrict__ anc8, int32_t *status_dev)
{
    // parent[] of this tree, staged once so that the root-path walks below run out of shared memory
    __shared__ int32_t par_s[GDN_MAX_TREE_NODES];
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
    for (int i = threadIdx.x; i < T; i += PLAN_THREADS) par_s[i] = parent[lo + i];
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
        }
        if (max_depth <= 16 && T <= 256)
            *reinterpret_cast<uint4 *>(anc8 + (size_t)(lo + i) * 16) = make_uint4(w0, w1, w2, w3);
    }
    const int any_err = __syncthreads_or(err != 0);
    if (err) report_status(status_dev, err);
    if (threadIdx.x == 0) tree_ok[b] = any_err ? 0 : 1;
}

}  // namespace

cudaError_t launch_plan(const gdn_shape_t &s, const int32_t *parent, const int32_t *node_offsets,
                        const PlanPtrs &plan, int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0) return cudaSuccess;
    plan_kernel<<<s.n_seq, PLAN_THREADS, 0, stream>>>(s.n_seq, s.total_nodes, s.max_tree_nodes,
                                                      s.max_depth, parent, node_offsets, plan.tree_ok,
                                                      plan.depth, plan.anc, plan.anc8, status_dev);
    return cudaGetLastError();
}

}  // namespace gdn
