// Tree metadata ("computed once per decode step", Section 3.4.2): for every node its depth and
// the list of nodes on its root path.  The ancestor sets of Section 3.4.2 are kept as explicit
// root-first lists rather than bitmasks: with at most max_depth (16 in the paper) nodes per path a
// list is smaller than a T-bit mask for T > 256 and lets the solve visit only real ancestors.
// Trees of more than 64 nodes additionally get a depth-first numbering cut into groups that are
// closed under "ancestor of" once the first node's root path is added (see gdn_internal.cuh); the
// tensor-core verify kernel takes one such group at a time.
#include "gdn_plan.cuh"

namespace gdn {

namespace {

__global__ void __launch_bounds__(PLAN_THREADS) plan_kernel(const PlanArgs a)
{
    // Programmatic stream serialization on both sides: this grid may have been launched under the tail of the
    // kernel in front of it (nothing is read before that kernel has completed), and the kernel behind this one
    // may be launched early in turn; it waits for this grid to finish before it reads anything written here.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    plan_tree(a, (int)blockIdx.x);
}

}  // namespace

cudaError_t launch_plan(const gdn_shape_t &s, const int32_t *parent, const int32_t *node_offsets,
                        const int32_t *n_nodes, const PlanPtrs &plan, int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0) return cudaSuccess;
    if (s.n_seq > 1) {   // the trees' CTAs claim their places in the unit list from a counter
        cudaError_t e0 = cudaMemsetAsync(plan.unit_count, 0, sizeof(int32_t), stream);
        if (e0 != cudaSuccess) return e0;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)s.n_seq);
    cfg.blockDim = dim3(PLAN_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, plan_kernel, plan_args(s, parent, node_offsets, n_nodes, plan, status_dev));
}

}  // namespace gdn
