// Internal declarations shared by the translation units of libgdn_tree.so.
// Nothing here is part of the public ABI (that is include/gdn_tree.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gdn_tree.h"

namespace gdn {

// Layout of the caller-provided verify workspace (all offsets 256-byte aligned).
//   tree_ok  int32 [n_seq]                 1 = tree passed the metadata checks
//   depth    uint8 [N]                     nodes on the root path of node n (root = 1)
//   anc      uint16[N][max_depth]          local ids of the root path of n, root first, n itself last
//   anc8     uint8 [N][16]                 the same list as bytes (filled when max_depth <= 16 and the
//                                          tree has <= 256 nodes; unused entries are 0xFF)
// Grouped verification of trees with more than 64 nodes (filled when max_depth <= 16 and the tree has at
// most GDN_GROUPED_MAX_NODES nodes).  "Position" = index in the depth-first pre-order of the tree (children
// by increasing id).  The positions are cut into consecutive groups; a group together with the proper
// ancestors of its first node (n_prefix <= 15 of them, all outside the group) is closed under "ancestor of", so it
// can be verified as a tree of its own: virtual index = depth-1 for those ancestors, n_prefix + offset in the
// group for the group's own nodes.  A group takes as many positions as the 64-node tile leaves after its prefix
// (64 - n_prefix, i.e. at least GDN_GROUP_MIN_NODES).
//   group_start uint16[n_seq][GDN_MAX_GROUPS + 1]  first position of group k of tree b; entries behind the
//                                          last group hold the tree's size
//   unit_count int32 [2]                   number of groups over all trees (zeroed in front of the plan kernel), and
//                                          a word that says for which shape the plan was built (plan_magic)
//   unit_list uint32[..][4]                one record per group, the groups of a tree next to one another, the trees
//                                          in the order in which their plan CTAs got there: (tree, first row of the
//                                          tree, first position | own nodes << 16, n_prefix | node at the first
//                                          position << 16).  A tree of at most 64 nodes is its own single group
//                                          (., ., T << 16, 0xFFFF): identity numbering, tables in depth / anc8.  The
//                                          tensor-core verify kernel walks this list, so that its units are real
//                                          groups only and spread evenly over the CTAs whatever the tree sizes.
//   dfs_node  uint16[N]                    node id at position r
//   dfs_depth uint8 [N]                    depth of that node
//   dfs_anc8  uint8 [N][16]                its root path in virtual indices of its group (0xFF = unused)
//   utilde   float [N][h_v][d_v]           solve result u~ (Eq. 10 with the W S0 term folded in; general kernel)
struct WorkspaceLayout {
    size_t tree_ok, depth, anc, anc8, dfs_node, dfs_depth, dfs_anc8, group_start, unit_count, unit_list, utilde, total;
};

constexpr int GDN_GROUP_TILE = 64;            // nodes of a group and its prefix together
constexpr int GDN_GROUP_MIN_NODES = 49;       // own nodes a group has at least (prefix of 15)
constexpr int GDN_GROUPED_MAX_NODES = 1024;   // largest tree the grouped tensor-core path takes
constexpr int GDN_MAX_GROUPS = (GDN_GROUPED_MAX_NODES + GDN_GROUP_MIN_NODES - 1) / GDN_GROUP_MIN_NODES;   // 21

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

// Written next to the unit count by the plan kernel and checked by the grouped verify kernel: a plan that was never
// built, or was built for another padded size, depth bound or number of trees, is refused instead of followed.
__host__ __device__ inline int32_t plan_magic(int n_trees, int max_tree_nodes, int max_depth)
{
    return (int32_t)(0x504C4E31u ^ ((uint32_t)n_trees * 2654435761u) ^ ((uint32_t)max_tree_nodes << 8) ^ (uint32_t)max_depth);
}
inline size_t unit_list_capacity(const gdn_shape_t &s)
{
    return (size_t)s.total_nodes / 49 + (size_t)s.n_seq + 1;
}

inline WorkspaceLayout workspace_layout(const gdn_shape_t &s)
{
    WorkspaceLayout w;
    size_t off = 0;
    const size_t N = (size_t)s.total_nodes;
    w.tree_ok = off;  off = align256(off + sizeof(int32_t) * (size_t)s.n_seq);
    w.depth = off;    off = align256(off + N);
    w.anc = off;      off = align256(off + sizeof(uint16_t) * N * (size_t)s.max_depth);
    w.anc8 = off;     off = align256(off + 16 * N);
    w.dfs_node = off; off = align256(off + 2 * N);
    w.dfs_depth = off; off = align256(off + N);
    w.dfs_anc8 = off; off = align256(off + 16 * N);
    w.group_start = off; off = align256(off + sizeof(uint16_t) * (size_t)s.n_seq * (GDN_MAX_GROUPS + 1));
    w.unit_count = off; off = align256(off + 2 * sizeof(int32_t));
    w.unit_list = off; off = align256(off + 16 * unit_list_capacity(s));
    w.utilde = off;   off = align256(off + sizeof(float) * N * (size_t)s.h_v * (size_t)s.d_v);
    w.total = off;
    return w;
}

struct PlanPtrs {
    int32_t *tree_ok;
    uint8_t *depth;
    uint16_t *anc;
    uint8_t *anc8;
    uint16_t *dfs_node;
    uint8_t *dfs_depth, *dfs_anc8;
    uint16_t *group_start;
    int32_t *unit_count;
    uint4 *unit_list;
    float *utilde;
};

inline PlanPtrs plan_ptrs(void *workspace, const WorkspaceLayout &w)
{
    char *b = static_cast<char *>(workspace);
    return {reinterpret_cast<int32_t *>(b + w.tree_ok), reinterpret_cast<uint8_t *>(b + w.depth),
            reinterpret_cast<uint16_t *>(b + w.anc), reinterpret_cast<uint8_t *>(b + w.anc8),
            reinterpret_cast<uint16_t *>(b + w.dfs_node), reinterpret_cast<uint8_t *>(b + w.dfs_depth),
            reinterpret_cast<uint8_t *>(b + w.dfs_anc8), reinterpret_cast<uint16_t *>(b + w.group_start),
            reinterpret_cast<int32_t *>(b + w.unit_count), reinterpret_cast<uint4 *>(b + w.unit_list),
            reinterpret_cast<float *>(b + w.utilde)};
}

// Host launchers (each returns the cudaError_t of its launch).
// node_offsets == nullptr: padded layout, s.n_seq trees of s.max_tree_nodes rows each (parent [n_seq][rows], the node
// counts in n_nodes [n_seq]); otherwise ragged packing and n_nodes is not read.
cudaError_t launch_plan(const gdn_shape_t &s, const int32_t *parent, const int32_t *node_offsets,
                        const int32_t *n_nodes, const PlanPtrs &plan, int32_t *status_dev, cudaStream_t stream);

cudaError_t launch_verify_generic(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                  const void *v, const void *g, const void *beta,
                                  const int32_t *node_offsets, void *o, const PlanPtrs &plan,
                                  cudaStream_t stream);

// Tensor-core fast path (d_k = d_v = 128, bf16 inputs, trees <= 64 nodes, root paths <= 16 nodes).
bool verify_sm100_supported(const gdn_shape_t &s);
bool verify_sm100_single_group(const gdn_shape_t &s);   // every tree fits one CTA (<= 64 nodes): fusable with commit
// Trees of at most 64 nodes: the kernel builds the tree metadata itself from parent[] (`plan` is not read);
// larger trees: `plan` must have been filled by launch_plan on the same stream.
cudaError_t launch_verify_sm100(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                const void *v, const void *g, const void *beta, const int32_t *parent,
                                const int32_t *node_offsets, void *o, const PlanPtrs &plan,
                                int32_t *status_dev, cudaStream_t stream);

// Same kernel with the commit of the previous step's accepted paths fused in front of the verify:
// the state tile is read once, advanced along the path (Eq. 7), written back, and the new tree is
// verified against the advanced state.
cudaError_t launch_commit_verify_sm100(const gdn_shape_t &s, float *S, const void *k_prev, const void *v_prev,
                                       const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                       const int32_t *node_offsets_prev, const int32_t *path,
                                       const int32_t *path_offsets, const void *q, const void *k, const void *v,
                                       const void *g, const void *beta, const int32_t *parent,
                                       const int32_t *node_offsets, void *o, int32_t *status_dev,
                                       cudaStream_t stream);

// Padded layout of Section 3.4.2 on the persistent tensor-core kernel (s.max_tree_nodes = rows per slot, s.total_nodes =
// n_seq * rows per slot, trees of at most 64 nodes): slot b carries tree b % n_trees; parent [n_trees][t_pad], n_nodes
// [n_trees]; raw_gates: g / beta are raw gate inputs.  The fused form takes the previous step in the same layout
// (prev_t_pad rows per slot) and one accepted path per tree: path [n_trees][max_depth], path_len [n_trees].
cudaError_t launch_verify_sm100_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, const float *S0,
                                       const void *q, const void *k, const void *v, const void *g, const void *beta,
                                       const int32_t *parent, const int32_t *n_nodes, void *o, int32_t *status_dev,
                                       cudaStream_t stream);
cudaError_t launch_commit_verify_sm100_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, float *S,
                                              int prev_t_pad, const void *k_prev, const void *v_prev,
                                              const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                              const int32_t *n_nodes_prev, const int32_t *path,
                                              const int32_t *path_len, const void *q, const void *k, const void *v,
                                              const void *g, const void *beta, const int32_t *parent,
                                              const int32_t *n_nodes, void *o, int32_t *status_dev,
                                              cudaStream_t stream);

// Padded layout, any padded tree size up to GDN_GROUPED_MAX_NODES: the plan of the n_trees shared trees (built by
// launch_plan with node_offsets == nullptr on a shape of n_trees trees) serves every slot; s.n_seq slots.
cudaError_t launch_verify_sm100_planned(const gdn_shape_t &s, int n_trees, bool raw_gates, const float *S0,
                                        const void *q, const void *k, const void *v, const void *g, const void *beta,
                                        const PlanPtrs &plan, void *o, int32_t *status_dev, cudaStream_t stream);

// Per-branch recurrent verification (the baseline of Section 5.2 / Figure 5): no workspace, no tree plan.
cudaError_t launch_verify_recurrent(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                    const void *v, const void *g, const void *beta, const int32_t *parent,
                                    const int32_t *node_offsets, void *o, int32_t *status_dev, cudaStream_t stream);

cudaError_t launch_commit_generic(const gdn_shape_t &s, float *S, const void *k, const void *v,
                                  const void *g, const void *beta, const int32_t *parent,
                                  const int32_t *node_offsets, const int32_t *path,
                                  const int32_t *path_offsets, int32_t *status_dev, cudaStream_t stream);
// d_k = d_v = 128, bf16 inputs, root paths of at most 16 nodes: the tile kernel's shapes.
bool commit_tile128_supported(const gdn_shape_t &s);
// The commit of the previous step's accepted paths (tile kernel, ragged packing) and the plan of the new trees in one
// grid: the fused call on trees of more than 64 nodes.  The new trees' shape is `s`; the commit reads only head counts
// and the depth bound from it.
cudaError_t launch_commit_plan(const gdn_shape_t &s, float *S, const void *k, const void *v, const void *g,
                               const void *beta, const int32_t *parent_prev, const int32_t *node_offsets_prev,
                               const int32_t *path, const int32_t *path_offsets, const int32_t *parent,
                               const int32_t *node_offsets, const PlanPtrs &plan, int32_t *status_dev,
                               cudaStream_t stream);
// Commit in the padded layout (d_k = d_v = 128, bf16, root paths of at most 16 nodes): slot b keeps its rows at
// b * s.max_tree_nodes and carries tree b % n_trees; parent [n_trees][rows] (may be null), n_nodes [n_trees],
// path [n_trees][s.max_depth], path_len [n_trees].
bool commit_padded_supported(const gdn_shape_t &s);
cudaError_t launch_commit_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, float *S, const void *k,
                                 const void *v, const void *g, const void *beta, const int32_t *parent,
                                 const int32_t *n_nodes, const int32_t *path, const int32_t *path_len,
                                 int32_t *status_dev, cudaStream_t stream);

#ifdef __CUDACC__
// First error wins; later ones are dropped.
__device__ __forceinline__ void report_status(int32_t *status_dev, int code)
{
    if (status_dev) atomicCAS(status_dev, 0, code);
}

// Gate activations of the "scalars" stage (Section 3.4.2; Table 1 row "scalars"): the kernel takes either the
// finished log-decay g and write strength beta, or the layer's raw gate inputs a, b, for which
// g = -softplus(a) = -log(1 + e^a) and beta = sigmoid(b) are formed here (fp32, never rounded to the input type).
__device__ __forceinline__ float gate_log_decay(uint32_t bf16_bits, bool raw)
{
    const float x = __uint_as_float(bf16_bits << 16);
    if (!raw) return x;
    return x > 0.f ? -(x + log1pf(expf(-x))) : -log1pf(expf(x));
}
__device__ __forceinline__ float gate_beta(uint32_t bf16_bits, bool raw)
{
    const float x = __uint_as_float(bf16_bits << 16);
    if (!raw) return x;
    const float e = expf(-fabsf(x));
    return x >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
}

template <typename T> __device__ __forceinline__ float load_as_float(const T *p);
template <> __device__ __forceinline__ float load_as_float<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16 *p)
{
    return __bfloat162float(__ldg(p));
}

template <typename T> __device__ __forceinline__ void store_from_float(T *p, float x);
template <> __device__ __forceinline__ void store_from_float<float>(float *p, float x) { *p = x; }
template <> __device__ __forceinline__ void store_from_float<__nv_bfloat16>(__nv_bfloat16 *p, float x)
{
    *p = __float2bfloat16_rn(x);
}
#endif

}  // namespace gdn
