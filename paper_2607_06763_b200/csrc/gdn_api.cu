// C-ABI entry points of libgdn_tree.so: argument validation, workspace carving, kernel launches,
// and the host-buffer variants.  See include/gdn_tree.h for the contract of every function.
#include <cstring>
#include <mutex>
#include <vector>

#include "gdn_internal.cuh"

using namespace gdn;

namespace {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t dtype_size(int dt) { return dt == GDN_BF16 ? 2 : 4; }

int check_shape(const gdn_shape_t *s)
{
    if (!s) return GDN_ERR_NULL;
    if (s->in_dtype != GDN_F32 && s->in_dtype != GDN_BF16) return GDN_ERR_DTYPE;
    if (s->out_dtype != GDN_F32 && s->out_dtype != GDN_BF16) return GDN_ERR_DTYPE;
    if (s->n_seq < 0 || s->h_qk < 1 || s->h_v < 1 || s->h_v % s->h_qk != 0) return GDN_ERR_SHAPE;
    if (s->d_k < 4 || s->d_k > GDN_MAX_HEAD_DIM || s->d_k % 4 != 0) return GDN_ERR_SHAPE;
    if (s->d_v < 1 || s->d_v > GDN_MAX_HEAD_DIM) return GDN_ERR_SHAPE;
    if (s->max_depth < 1 || s->max_depth > GDN_MAX_DEPTH_CAP) return GDN_ERR_SHAPE;
    if (s->total_nodes < 0 || s->max_tree_nodes < 1 || s->max_tree_nodes > GDN_MAX_TREE_NODES)
        return GDN_ERR_SHAPE;
    if ((long long)s->n_seq * s->h_v > 0x7fffffffLL) return GDN_ERR_SHAPE;
    if (!(s->scale == s->scale)) return GDN_ERR_SHAPE;   // NaN
    // rows of q/k/v must keep 16-byte alignment of the tensor bases meaningful for vector loads
    if ((s->d_k * dtype_size(s->in_dtype)) % 8 != 0) return GDN_ERR_SHAPE;
    return GDN_OK;
}

struct TensorBytes {
    size_t state, qk, v, gb, o, parent, offsets;
};

TensorBytes tensor_bytes(const gdn_shape_t &s)
{
    const size_t N = (size_t)s.total_nodes, isz = dtype_size(s.in_dtype), osz = dtype_size(s.out_dtype);
    TensorBytes t;
    t.state = (size_t)s.n_seq * s.h_v * s.d_v * s.d_k * sizeof(float);
    t.qk = N * s.h_qk * s.d_k * isz;
    t.v = N * s.h_v * s.d_v * isz;
    t.gb = N * s.h_v * isz;
    t.o = N * s.h_v * s.d_v * osz;
    t.parent = N * sizeof(int32_t);
    t.offsets = ((size_t)s.n_seq + 1) * sizeof(int32_t);
    return t;
}

// Bump allocator over the caller's device arena (host-buffer entry points).
struct Arena {
    char *base;
    size_t off, cap;
    void *take(size_t bytes)
    {
        void *p = base + off;
        off = align256(off + bytes);
        return off <= cap ? p : nullptr;
    }
};

// Host-side argument checks of gdn_tree_verify (everything that can be refused before a launch).
int check_verify_args(const gdn_shape_t &s, const float *S0, const void *q, const void *k, const void *v,
                      const void *g, const void *beta, const int32_t *parent, const int32_t *node_offsets,
                      const void *o, const void *workspace, size_t workspace_bytes, const int32_t *status_dev)
{
    if (!S0 || !q || !k || !v || !g || !beta || !parent || !node_offsets || !o || !status_dev)
        return GDN_ERR_NULL;
    if (!workspace) return GDN_ERR_WORKSPACE;
    if (!aligned16(S0) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) ||
        !aligned16(beta) || !aligned16(o) || !aligned256(workspace) ||
        (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(node_offsets) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    if (workspace_bytes < workspace_layout(s).total) return GDN_ERR_WORKSPACE;
    return GDN_OK;
}

// Host-side argument checks of gdn_tree_commit.
int check_commit_args(const gdn_shape_t &s, const float *S, const void *k, const void *v, const void *g,
                      const void *beta, const int32_t *parent, const int32_t *node_offsets, const int32_t *path,
                      const int32_t *path_offsets, const int32_t *status_dev)
{
    if (!S || !node_offsets || !path_offsets || !status_dev) return GDN_ERR_NULL;
    if (s.total_nodes > 0 && (!k || !v || !g || !beta || !path)) return GDN_ERR_NULL;
    if (!aligned16(S) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(node_offsets) & 3u) ||
        (reinterpret_cast<uintptr_t>(path) & 3u) || (reinterpret_cast<uintptr_t>(path_offsets) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    return GDN_OK;
}

}  // namespace

extern "C" const char *gdn_status_string(int status)
{
    switch (status) {
    case GDN_OK: return "ok";
    case GDN_ERR_NULL: return "a required pointer is NULL";
    case GDN_ERR_SHAPE: return "a size is out of range or inconsistent";
    case GDN_ERR_DTYPE: return "unknown dtype";
    case GDN_ERR_ALIGN: return "a pointer is not aligned as required";
    case GDN_ERR_UNSUPPORTED: return "request not supported by this build";
    case GDN_ERR_CUDA: return "a CUDA runtime call failed";
    case GDN_ERR_TREE: return "parent[]/node_offsets[] do not describe a topological forest";
    case GDN_ERR_DEPTH: return "a root path has more than max_depth nodes";
    case GDN_ERR_PATH: return "accepted path is not a root chain of its tree";
    case GDN_ERR_WORKSPACE: return "workspace missing or too small";
    case GDN_ERR_TIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
    }
}

extern "C" size_t gdn_tree_workspace_bytes(const gdn_shape_t *shape)
{
    if (check_shape(shape) != GDN_OK) return 0;
    return workspace_layout(*shape).total;
}

extern "C" int gdn_tree_validate_host(const gdn_shape_t *shape, const int32_t *parent_h,
                                      const int32_t *node_offsets_h, const int32_t *path_h,
                                      const int32_t *path_offsets_h)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    if (!node_offsets_h || (!parent_h && shape->total_nodes > 0)) return GDN_ERR_NULL;
    if ((path_h == nullptr) != (path_offsets_h == nullptr) && path_offsets_h == nullptr) return GDN_ERR_NULL;
    const gdn_shape_t &s = *shape;
    if (node_offsets_h[0] != 0 || node_offsets_h[s.n_seq] != s.total_nodes) return GDN_ERR_TREE;
    for (int b = 0; b < s.n_seq; ++b) {
        const int lo = node_offsets_h[b], T = node_offsets_h[b + 1] - lo;
        if (T < 0 || T > s.max_tree_nodes) return GDN_ERR_TREE;
    }
    // depth of every node by one forward pass (parents come first)
    int worst = GDN_OK;
    for (int b = 0; b < s.n_seq && worst == GDN_OK; ++b) {
        const int lo = node_offsets_h[b], T = node_offsets_h[b + 1] - lo;
        for (int i = 0; i < T; ++i) {
            const int p = parent_h[lo + i];
            if (p < -1 || p >= i) return GDN_ERR_TREE;
        }
        for (int i = 0; i < T; ++i) {
            int d = 0;
            for (int cur = i; cur >= 0; cur = parent_h[lo + cur])
                if (++d > s.max_depth) return GDN_ERR_DEPTH;
        }
    }
    if (path_offsets_h) {
        if (path_offsets_h[0] != 0) return GDN_ERR_PATH;
        for (int b = 0; b < s.n_seq; ++b) {
            const int lo = node_offsets_h[b], T = node_offsets_h[b + 1] - lo;
            const int p0 = path_offsets_h[b], L = path_offsets_h[b + 1] - p0;
            if (L < 0 || L > s.max_depth) return GDN_ERR_PATH;
            if (L > 0 && !path_h) return GDN_ERR_NULL;
            for (int t = 0; t < L; ++t) {
                const int n = path_h[p0 + t];
                if (n < 0 || n >= T) return GDN_ERR_PATH;
                if (parent_h[lo + n] != (t ? path_h[p0 + t - 1] : -1)) return GDN_ERR_PATH;
            }
        }
    }
    return worst;
}

extern "C" int gdn_tree_verify(const gdn_shape_t *shape, const float *S0, const void *q, const void *k,
                               const void *v, const void *g, const void *beta, const int32_t *parent,
                               const int32_t *node_offsets, void *o, void *workspace,
                               size_t workspace_bytes, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    rc = check_verify_args(s, S0, q, k, v, g, beta, parent, node_offsets, o, workspace, workspace_bytes, status_dev);
    if (rc != GDN_OK) return rc;
    const WorkspaceLayout lay = workspace_layout(s);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const PlanPtrs plan = plan_ptrs(workspace, lay);
    // trees of at most 64 nodes on the tensor-core path: that kernel builds the tree metadata itself
    if (!verify_sm100_single_group(s) &&
        launch_plan(s, parent, node_offsets, nullptr, plan, status_dev, stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    const cudaError_t e = verify_sm100_supported(s)
                              ? launch_verify_sm100(s, S0, q, k, v, g, beta, parent, node_offsets, o, plan, status_dev, stream)
                              : launch_verify_generic(s, S0, q, k, v, g, beta, node_offsets, o, plan, stream);
    if (e != cudaSuccess) return GDN_ERR_CUDA;
    return GDN_OK;
}

namespace {

// Shape rules of the padded entry points: rows per slot = max_tree_nodes, total_nodes = n_seq * rows, every tree
// shared by n_seq / n_trees slots; they run on the persistent tensor-core kernel only.
int check_padded_shape(const gdn_shape_t &s, int32_t n_trees)
{
    if (n_trees < 1 || s.n_seq % n_trees != 0) return GDN_ERR_SHAPE;
    if ((long long)s.n_seq * s.max_tree_nodes != s.total_nodes) return GDN_ERR_SHAPE;
    if (!verify_sm100_single_group(s)) return GDN_ERR_UNSUPPORTED;
    return GDN_OK;
}

}  // namespace

extern "C" int gdn_tree_verify_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, const float *S0,
                                      const void *q, const void *k, const void *v, const void *g, const void *beta,
                                      const int32_t *parent, const int32_t *n_nodes, void *o, int32_t *status_dev,
                                      void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    rc = check_padded_shape(s, n_trees);
    if (rc != GDN_OK) return rc;
    if (!S0 || !q || !k || !v || !g || !beta || !parent || !n_nodes || !o || !status_dev) return GDN_ERR_NULL;
    if (!aligned16(S0) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(o) || (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(n_nodes) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    if (launch_verify_sm100_padded(s, n_trees, raw_gates != 0, S0, q, k, v, g, beta, parent, n_nodes, o, status_dev,
                                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_commit_verify_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, float *S,
                                             int32_t prev_t_pad, const void *k_prev, const void *v_prev,
                                             const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                             const int32_t *n_nodes_prev, const int32_t *path,
                                             const int32_t *path_len, const void *q, const void *k, const void *v,
                                             const void *g, const void *beta, const int32_t *parent,
                                             const int32_t *n_nodes, void *o, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    rc = check_padded_shape(s, n_trees);
    if (rc != GDN_OK) return rc;
    if (prev_t_pad < 1 || prev_t_pad > GDN_MAX_TREE_NODES) return GDN_ERR_SHAPE;
    if (!S || !k_prev || !v_prev || !g_prev || !beta_prev || !n_nodes_prev || !path || !path_len || !q || !k || !v ||
        !g || !beta || !parent || !n_nodes || !o || !status_dev)
        return GDN_ERR_NULL;
    if (!aligned16(S) || !aligned16(k_prev) || !aligned16(v_prev) || !aligned16(g_prev) || !aligned16(beta_prev) ||
        !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) || !aligned16(o) ||
        (reinterpret_cast<uintptr_t>(parent_prev) & 3u) || (reinterpret_cast<uintptr_t>(n_nodes_prev) & 3u) ||
        (reinterpret_cast<uintptr_t>(path) & 3u) || (reinterpret_cast<uintptr_t>(path_len) & 3u) ||
        (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(n_nodes) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    if (launch_commit_verify_sm100_padded(s, n_trees, raw_gates != 0, S, prev_t_pad, k_prev, v_prev, g_prev, beta_prev,
                                          parent_prev, n_nodes_prev, path, path_len, q, k, v, g, beta, parent, n_nodes,
                                          o, status_dev, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

namespace {

// The shared-tree plan of the padded layout: the tree-metadata part of the verify workspace for n_trees trees of
// shape.max_tree_nodes rows each (no u~ buffer).
gdn_shape_t plan_shape(const gdn_shape_t &s, int32_t n_trees)
{
    gdn_shape_t ps = s;
    ps.n_seq = n_trees;
    ps.total_nodes = n_trees * s.max_tree_nodes;
    ps.h_v = 0;   // sizes the u~ buffer of the general verify kernel, which the plan does not have
    return ps;
}

int check_planned_shape(const gdn_shape_t &s, int32_t n_trees)
{
    if (n_trees < 1 || s.n_seq % n_trees != 0) return GDN_ERR_SHAPE;
    if ((long long)s.n_seq * s.max_tree_nodes != s.total_nodes) return GDN_ERR_SHAPE;
    if (!verify_sm100_supported(s)) return GDN_ERR_UNSUPPORTED;
    return GDN_OK;
}

}  // namespace

extern "C" size_t gdn_tree_plan_bytes(const gdn_shape_t *shape, int32_t n_trees)
{
    if (check_shape(shape) != GDN_OK || n_trees < 1) return 0;
    return workspace_layout(plan_shape(*shape, n_trees)).total;
}

extern "C" int gdn_tree_plan(const gdn_shape_t *shape, int32_t n_trees, const int32_t *parent, const int32_t *n_nodes,
                             void *plan, size_t plan_bytes, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    rc = check_planned_shape(s, n_trees);
    if (rc != GDN_OK) return rc;
    if (!parent || !n_nodes || !status_dev) return GDN_ERR_NULL;
    if (!plan) return GDN_ERR_WORKSPACE;
    if (!aligned256(plan) || (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(n_nodes) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    const gdn_shape_t ps = plan_shape(s, n_trees);
    const WorkspaceLayout lay = workspace_layout(ps);
    if (plan_bytes < lay.total) return GDN_ERR_WORKSPACE;
    if (launch_plan(ps, parent, nullptr, n_nodes, plan_ptrs(plan, lay), status_dev,
                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_verify_planned(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, const float *S0,
                                       const void *q, const void *k, const void *v, const void *g, const void *beta,
                                       const void *plan, size_t plan_bytes, void *o, int32_t *status_dev,
                                       void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    rc = check_planned_shape(s, n_trees);
    if (rc != GDN_OK) return rc;
    if (!S0 || !q || !k || !v || !g || !beta || !o || !status_dev) return GDN_ERR_NULL;
    if (!plan) return GDN_ERR_WORKSPACE;
    if (!aligned16(S0) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(o) || !aligned256(plan) || (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    const WorkspaceLayout lay = workspace_layout(plan_shape(s, n_trees));
    if (plan_bytes < lay.total) return GDN_ERR_WORKSPACE;
    if (launch_verify_sm100_planned(s, n_trees, raw_gates != 0, S0, q, k, v, g, beta,
                                    plan_ptrs(const_cast<void *>(plan), lay), o, status_dev,
                                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_commit_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, float *S,
                                      const void *k, const void *v, const void *g, const void *beta,
                                      const int32_t *parent, const int32_t *n_nodes, const int32_t *path,
                                      const int32_t *path_len, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    if (n_trees < 1 || s.n_seq % n_trees != 0) return GDN_ERR_SHAPE;
    if ((long long)s.n_seq * s.max_tree_nodes != s.total_nodes) return GDN_ERR_SHAPE;
    if (!commit_padded_supported(s)) return GDN_ERR_UNSUPPORTED;
    if (!S || !k || !v || !g || !beta || !n_nodes || !path || !path_len || !status_dev) return GDN_ERR_NULL;
    if (!aligned16(S) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        (reinterpret_cast<uintptr_t>(parent) & 3u) || (reinterpret_cast<uintptr_t>(n_nodes) & 3u) ||
        (reinterpret_cast<uintptr_t>(path) & 3u) || (reinterpret_cast<uintptr_t>(path_len) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    if (launch_commit_padded(s, n_trees, raw_gates != 0, S, k, v, g, beta, parent, n_nodes, path, path_len, status_dev,
                             static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_verify_recurrent(const gdn_shape_t *shape, const float *S0, const void *q, const void *k,
                                         const void *v, const void *g, const void *beta, const int32_t *parent,
                                         const int32_t *node_offsets, void *o, int32_t *status_dev,
                                         void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    if (!S0 || !q || !k || !v || !g || !beta || !parent || !node_offsets || !o || !status_dev) return GDN_ERR_NULL;
    if (!aligned16(S0) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(o) || (reinterpret_cast<uintptr_t>(parent) & 3u) ||
        (reinterpret_cast<uintptr_t>(node_offsets) & 3u) || (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    if (launch_verify_recurrent(s, S0, q, k, v, g, beta, parent, node_offsets, o, status_dev,
                                static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_commit(const gdn_shape_t *shape, float *S, const void *k, const void *v,
                               const void *g, const void *beta, const int32_t *parent,
                               const int32_t *node_offsets, const int32_t *path,
                               const int32_t *path_offsets, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0) return GDN_OK;
    rc = check_commit_args(s, S, k, v, g, beta, parent, node_offsets, path, path_offsets, status_dev);
    if (rc != GDN_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (launch_commit_generic(s, S, k, v, g, beta, parent, node_offsets, path, path_offsets, status_dev,
                              stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" int gdn_tree_commit_verify(const gdn_shape_t *shape, float *S, const void *k_prev, const void *v_prev,
                                      const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                      const int32_t *node_offsets_prev, const int32_t *path,
                                      const int32_t *path_offsets, const void *q, const void *k, const void *v,
                                      const void *g, const void *beta, const int32_t *parent,
                                      const int32_t *node_offsets, void *o, void *workspace,
                                      size_t workspace_bytes, int32_t *status_dev, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0) return GDN_OK;
    if (!S || !node_offsets_prev || !path_offsets || !status_dev) return GDN_ERR_NULL;
    if (!verify_sm100_single_group(s) || s.total_nodes == 0) {
        // general shapes: the two kernels back to back on the stream (the shape's node counts are
        // not used by commit, so the new tree's shape serves for the previous tree as well).  Both
        // halves are checked before the first launch: a refused call must leave the state as it was.
        rc = check_commit_args(s, S, k_prev, v_prev, g_prev, beta_prev, parent_prev, node_offsets_prev, path,
                               path_offsets, status_dev);
        if (rc != GDN_OK) return rc;
        if (s.total_nodes > 0) {
            rc = check_verify_args(s, S, q, k, v, g, beta, parent, node_offsets, o, workspace, workspace_bytes,
                                   status_dev);
            if (rc != GDN_OK) return rc;
        }
        if (s.total_nodes > 0 && verify_sm100_supported(s) && commit_tile128_supported(s)) {
            // trees of more than 64 nodes on the tensor-core path: the plan of the new trees does not depend on the
            // commit, so it is built by extra CTAs of the commit grid; then the verify kernel in its grouped mode
            const WorkspaceLayout lay = workspace_layout(s);
            const PlanPtrs plan = plan_ptrs(workspace, lay);
            cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
            if (launch_commit_plan(s, S, k_prev, v_prev, g_prev, beta_prev, parent_prev, node_offsets_prev, path,
                                   path_offsets, parent, node_offsets, plan, status_dev, stream) != cudaSuccess)
                return GDN_ERR_CUDA;
            if (launch_verify_sm100(s, S, q, k, v, g, beta, parent, node_offsets, o, plan, status_dev, stream) !=
                cudaSuccess)
                return GDN_ERR_CUDA;
            return GDN_OK;
        }
        rc = gdn_tree_commit(shape, S, k_prev, v_prev, g_prev, beta_prev, parent_prev, node_offsets_prev, path,
                             path_offsets, status_dev, cuda_stream);
        if (rc != GDN_OK) return rc;
        return gdn_tree_verify(shape, S, q, k, v, g, beta, parent, node_offsets, o, workspace, workspace_bytes,
                               status_dev, cuda_stream);
    }
    if (!k_prev || !v_prev || !g_prev || !beta_prev || !path) return GDN_ERR_NULL;
    if (!q || !k || !v || !g || !beta || !parent || !node_offsets || !o) return GDN_ERR_NULL;
    if (!workspace) return GDN_ERR_WORKSPACE;
    if (!aligned16(S) || !aligned16(k_prev) || !aligned16(v_prev) || !aligned16(g_prev) || !aligned16(beta_prev) ||
        !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) || !aligned16(o) ||
        !aligned256(workspace) || (reinterpret_cast<uintptr_t>(parent_prev) & 3u) ||
        (reinterpret_cast<uintptr_t>(node_offsets_prev) & 3u) || (reinterpret_cast<uintptr_t>(path) & 3u) ||
        (reinterpret_cast<uintptr_t>(path_offsets) & 3u) || (reinterpret_cast<uintptr_t>(parent) & 3u) ||
        (reinterpret_cast<uintptr_t>(node_offsets) & 3u) || (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return GDN_ERR_ALIGN;
    const WorkspaceLayout lay = workspace_layout(s);
    if (workspace_bytes < lay.total) return GDN_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (launch_commit_verify_sm100(s, S, k_prev, v_prev, g_prev, beta_prev, parent_prev, node_offsets_prev, path,
                                   path_offsets, q, k, v, g, beta, parent, node_offsets, o, status_dev,
                                   stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

extern "C" size_t gdn_tree_host_arena_bytes(const gdn_shape_t *shape, int32_t total_path_len)
{
    if (check_shape(shape) != GDN_OK || total_path_len < 0) return 0;
    const TensorBytes t = tensor_bytes(*shape);
    size_t n = 0;
    n += align256(t.state) + 2 * align256(t.qk) + align256(t.v) + 2 * align256(t.gb) + align256(t.o);
    n += align256(t.parent) + 2 * align256(t.offsets) + align256((size_t)total_path_len * sizeof(int32_t) + 4);
    n += align256(sizeof(int32_t));            // status word
    n += workspace_layout(*shape).total;       // verify workspace
    return n + 256;
}

#define GDN_CUDA_TRY(expr)                         \
    do {                                           \
        if ((expr) != cudaSuccess) return GDN_ERR_CUDA; \
    } while (0)

extern "C" int gdn_tree_verify_host(const gdn_shape_t *shape, const float *S0_h, const void *q_h,
                                    const void *k_h, const void *v_h, const void *g_h,
                                    const void *beta_h, const int32_t *parent_h,
                                    const int32_t *node_offsets_h, void *o_h, void *dev_arena,
                                    size_t arena_bytes, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || s.total_nodes == 0) return GDN_OK;
    if (!S0_h || !q_h || !k_h || !v_h || !g_h || !beta_h || !parent_h || !node_offsets_h || !o_h)
        return GDN_ERR_NULL;
    if (!dev_arena || arena_bytes < gdn_tree_host_arena_bytes(shape, 0)) return GDN_ERR_WORKSPACE;
    if (!aligned256(dev_arena)) return GDN_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const TensorBytes t = tensor_bytes(s);
    Arena a{static_cast<char *>(dev_arena), 0, arena_bytes};
    float *S0 = static_cast<float *>(a.take(t.state));
    void *q = a.take(t.qk), *k = a.take(t.qk), *v = a.take(t.v), *g = a.take(t.gb), *beta = a.take(t.gb);
    void *o = a.take(t.o);
    int32_t *parent = static_cast<int32_t *>(a.take(t.parent));
    int32_t *offs = static_cast<int32_t *>(a.take(t.offsets));
    int32_t *status = static_cast<int32_t *>(a.take(sizeof(int32_t)));
    const size_t ws_bytes = workspace_layout(s).total;
    void *ws = a.take(ws_bytes);
    if (!ws) return GDN_ERR_WORKSPACE;
    GDN_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(S0, S0_h, t.state, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(q, q_h, t.qk, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(k, k_h, t.qk, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(v, v_h, t.v, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(g, g_h, t.gb, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(beta, beta_h, t.gb, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(parent, parent_h, t.parent, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(offs, node_offsets_h, t.offsets, cudaMemcpyHostToDevice, stream));
    rc = gdn_tree_verify(shape, S0, q, k, v, g, beta, parent, offs, o, ws, ws_bytes, status, cuda_stream);
    if (rc != GDN_OK) return rc;
    int32_t status_h = 0;
    GDN_CUDA_TRY(cudaMemcpyAsync(o_h, o, t.o, cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(&status_h, status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaStreamSynchronize(stream));
    return status_h;
}

extern "C" int gdn_tree_commit_host(const gdn_shape_t *shape, float *S_h, const void *k_h,
                                    const void *v_h, const void *g_h, const void *beta_h,
                                    const int32_t *parent_h, const int32_t *node_offsets_h,
                                    const int32_t *path_h, const int32_t *path_offsets_h,
                                    int32_t total_path_len, void *dev_arena, size_t arena_bytes,
                                    void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0 || total_path_len == 0) return GDN_OK;
    if (total_path_len < 0) return GDN_ERR_SHAPE;
    if (!S_h || !k_h || !v_h || !g_h || !beta_h || !node_offsets_h || !path_h || !path_offsets_h)
        return GDN_ERR_NULL;
    if (!dev_arena || arena_bytes < gdn_tree_host_arena_bytes(shape, total_path_len)) return GDN_ERR_WORKSPACE;
    if (!aligned256(dev_arena)) return GDN_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const TensorBytes t = tensor_bytes(s);
    Arena a{static_cast<char *>(dev_arena), 0, arena_bytes};
    float *S = static_cast<float *>(a.take(t.state));
    void *k = a.take(t.qk), *v = a.take(t.v), *g = a.take(t.gb), *beta = a.take(t.gb);
    int32_t *parent = parent_h ? static_cast<int32_t *>(a.take(t.parent)) : nullptr;
    int32_t *offs = static_cast<int32_t *>(a.take(t.offsets));
    int32_t *poffs = static_cast<int32_t *>(a.take(t.offsets));
    const size_t path_bytes = (size_t)total_path_len * sizeof(int32_t);
    int32_t *path = static_cast<int32_t *>(a.take(path_bytes));
    int32_t *status = static_cast<int32_t *>(a.take(sizeof(int32_t)));
    if (!status) return GDN_ERR_WORKSPACE;
    GDN_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(S, S_h, t.state, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(k, k_h, t.qk, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(v, v_h, t.v, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(g, g_h, t.gb, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(beta, beta_h, t.gb, cudaMemcpyHostToDevice, stream));
    if (parent) GDN_CUDA_TRY(cudaMemcpyAsync(parent, parent_h, t.parent, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(offs, node_offsets_h, t.offsets, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(poffs, path_offsets_h, t.offsets, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(path, path_h, path_bytes, cudaMemcpyHostToDevice, stream));
    rc = gdn_tree_commit(shape, S, k, v, g, beta, parent, offs, path, poffs, status, cuda_stream);
    if (rc != GDN_OK) return rc;
    int32_t status_h = 0;
    GDN_CUDA_TRY(cudaMemcpyAsync(S_h, S, t.state, cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(&status_h, status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaStreamSynchronize(stream));
    return status_h;
}

namespace {

// Helper streams and events of the pipelined host-buffer call, created on first use for each device and kept for
// the life of the process (the one piece of state the library keeps besides the static scratch array).
constexpr int HOST_PIPE_GROUPS = 6;
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, in[HOST_PIPE_GROUPS] = {}, k[HOST_PIPE_GROUPS] = {};
};
std::mutex g_pipe_mutex;
HostPipe g_pipe[64];

HostPipe *host_pipe()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe &p = g_pipe[dev];
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < HOST_PIPE_GROUPS; ++i)
            ok = cudaEventCreateWithFlags(&p.in[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.k[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        p.ready = true;
    }
    return &p;
}

}  // namespace

extern "C" size_t gdn_tree_commit_verify_host_arena_bytes(const gdn_shape_t *shape, int32_t prev_total_nodes,
                                                          int32_t total_path_len)
{
    if (check_shape(shape) != GDN_OK || total_path_len < 0 || prev_total_nodes < 0) return 0;
    gdn_shape_t prev = *shape;
    prev.total_nodes = prev_total_nodes;
    const TensorBytes t = tensor_bytes(*shape), tp = tensor_bytes(prev);
    size_t n = 0;
    n += align256(t.state) + 2 * align256(t.qk) + align256(t.v) + 2 * align256(t.gb) + align256(t.o);
    n += align256(t.parent) + align256(t.offsets);
    n += align256(tp.qk) + align256(tp.v) + 2 * align256(tp.gb) + align256(tp.parent) + 2 * align256(tp.offsets);
    n += align256((size_t)total_path_len * sizeof(int32_t) + 4) + align256(sizeof(int32_t));
    n += workspace_layout(*shape).total;
    n += 3 * align256(sizeof(int32_t) * ((size_t)shape->n_seq + HOST_PIPE_GROUPS + 1));   // per-group offset arrays
    return n + 256;
}

extern "C" int gdn_tree_commit_verify_host(const gdn_shape_t *shape, float *S_h, int32_t prev_total_nodes,
                                           const void *k_prev_h, const void *v_prev_h, const void *g_prev_h,
                                           const void *beta_prev_h, const int32_t *parent_prev_h,
                                           const int32_t *node_offsets_prev_h, const int32_t *path_h,
                                           const int32_t *path_offsets_h, int32_t total_path_len, const void *q_h,
                                           const void *k_h, const void *v_h, const void *g_h, const void *beta_h,
                                           const int32_t *parent_h, const int32_t *node_offsets_h, void *o_h,
                                           void *dev_arena, size_t arena_bytes, void *cuda_stream)
{
    int rc = check_shape(shape);
    if (rc != GDN_OK) return rc;
    const gdn_shape_t &s = *shape;
    if (s.n_seq == 0) return GDN_OK;
    if (total_path_len < 0 || prev_total_nodes < 0) return GDN_ERR_SHAPE;
    if (!S_h || !node_offsets_prev_h || !path_offsets_h || !node_offsets_h) return GDN_ERR_NULL;
    if (total_path_len > 0 && (!k_prev_h || !v_prev_h || !g_prev_h || !beta_prev_h || !path_h)) return GDN_ERR_NULL;
    if (s.total_nodes > 0 && (!q_h || !k_h || !v_h || !g_h || !beta_h || !parent_h || !o_h)) return GDN_ERR_NULL;
    if (!dev_arena || arena_bytes < gdn_tree_commit_verify_host_arena_bytes(shape, prev_total_nodes, total_path_len))
        return GDN_ERR_WORKSPACE;
    if (!aligned256(dev_arena)) return GDN_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    gdn_shape_t prev = s;
    prev.total_nodes = prev_total_nodes;
    const TensorBytes t = tensor_bytes(s), tp = tensor_bytes(prev);
    const WorkspaceLayout lay = workspace_layout(s);
    Arena a{static_cast<char *>(dev_arena), 0, arena_bytes};
    float *S = static_cast<float *>(a.take(t.state));
    void *q = a.take(t.qk), *k = a.take(t.qk), *v = a.take(t.v), *g = a.take(t.gb), *beta = a.take(t.gb);
    void *o = a.take(t.o);
    int32_t *parent = static_cast<int32_t *>(a.take(t.parent));
    int32_t *offs = static_cast<int32_t *>(a.take(t.offsets));
    void *kp = a.take(tp.qk), *vp = a.take(tp.v), *gp = a.take(tp.gb), *bp = a.take(tp.gb);
    int32_t *parent_p = parent_prev_h ? static_cast<int32_t *>(a.take(tp.parent)) : nullptr;
    int32_t *offs_p = static_cast<int32_t *>(a.take(tp.offsets));
    int32_t *poffs = static_cast<int32_t *>(a.take(tp.offsets));
    const size_t path_bytes = (size_t)total_path_len * sizeof(int32_t);
    int32_t *path = static_cast<int32_t *>(a.take(path_bytes + 4));
    int32_t *status = static_cast<int32_t *>(a.take(sizeof(int32_t)));
    void *ws = a.take(lay.total);
    const size_t goff_bytes = sizeof(int32_t) * ((size_t)s.n_seq + HOST_PIPE_GROUPS + 1);
    int32_t *g_offs = static_cast<int32_t *>(a.take(goff_bytes));
    int32_t *g_offs_p = static_cast<int32_t *>(a.take(goff_bytes));
    int32_t *g_poffs = static_cast<int32_t *>(a.take(goff_bytes));
    if (!ws || !g_poffs) return GDN_ERR_WORKSPACE;
    GDN_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), stream));
    // group slices of g / beta start at multiples of h_v elements: they keep the 16-byte alignment the device entry
    // points ask for only if a row of them is a multiple of 16 bytes (otherwise the call runs unpipelined)
    const bool sliceable = ((size_t)s.h_v * dtype_size(s.in_dtype)) % 16 == 0;
    HostPipe *pipe = (sliceable && s.n_seq >= 2 && s.total_nodes > 0 && total_path_len > 0) ? host_pipe() : nullptr;
    if (pipe) {
        // Pipelined form: the layer slots / sequences are cut into groups; the copies up of group i+1 (helper stream
        // s_in), the kernels of group i (the caller's stream) and the copies down of group i-1 (helper stream s_out)
        // run at the same time, so that both directions of the host link are busy.  Each group is a call of its own
        // on slices of the packed tensors, with node and path offsets rebased to its first row.
        const int G = s.n_seq < HOST_PIPE_GROUPS ? s.n_seq : HOST_PIPE_GROUPS;
        std::vector<int32_t> ho((size_t)s.n_seq + G), hop((size_t)s.n_seq + G), hpo((size_t)s.n_seq + G);
        std::vector<int> first(G + 1);
        for (int i = 0; i <= G; ++i) first[i] = (int)((long long)s.n_seq * i / G);
        for (int i = 0; i < G; ++i)
            for (int b = first[i]; b <= first[i + 1]; ++b) {
                ho[(size_t)b + i] = node_offsets_h[b] - node_offsets_h[first[i]];
                hop[(size_t)b + i] = node_offsets_prev_h[b] - node_offsets_prev_h[first[i]];
                hpo[(size_t)b + i] = path_offsets_h[b] - path_offsets_h[first[i]];
            }
        const size_t ob = sizeof(int32_t) * ho.size();
        GDN_CUDA_TRY(cudaMemcpyAsync(g_offs, ho.data(), ob, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(g_offs_p, hop.data(), ob, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(g_poffs, hpo.data(), ob, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaEventRecord(pipe->start, stream));
        GDN_CUDA_TRY(cudaStreamWaitEvent(pipe->s_in, pipe->start, 0));
        GDN_CUDA_TRY(cudaStreamWaitEvent(pipe->s_out, pipe->start, 0));
        const size_t isz = dtype_size(s.in_dtype), osz = dtype_size(s.out_dtype);
        const size_t row_qk = (size_t)s.h_qk * s.d_k * isz, row_v = (size_t)s.h_v * s.d_v * isz, row_gb = (size_t)s.h_v * isz;
        const size_t row_o = (size_t)s.h_v * s.d_v * osz, slot_state = (size_t)s.h_v * s.d_v * s.d_k * sizeof(float);
        auto at = [](const void *base, size_t off) { return static_cast<const char *>(base) + off; };
        auto atw = [](void *base, size_t off) { return static_cast<char *>(base) + off; };
        // the small tensors (gates, trees, paths: a percent of the bytes) go up whole in front of the first group: a
        // copy costs a few microseconds whatever its size, and per group only the large slices are left
        {
            cudaStream_t si = pipe->s_in;
            GDN_CUDA_TRY(cudaMemcpyAsync(g, g_h, t.gb, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(beta, beta_h, t.gb, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(parent, parent_h, t.parent, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(gp, g_prev_h, tp.gb, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(bp, beta_prev_h, tp.gb, cudaMemcpyHostToDevice, si));
            if (parent_p) GDN_CUDA_TRY(cudaMemcpyAsync(parent_p, parent_prev_h, tp.parent, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(path, path_h, path_bytes, cudaMemcpyHostToDevice, si));
        }
        for (int i = 0; i < G; ++i) {
            const int b0 = first[i], nb = first[i + 1] - b0;
            const size_t n0 = (size_t)node_offsets_h[b0], nn = (size_t)node_offsets_h[b0 + nb] - n0;
            const size_t m0 = (size_t)node_offsets_prev_h[b0], mm = (size_t)node_offsets_prev_h[b0 + nb] - m0;
            const size_t p0 = (size_t)path_offsets_h[b0], pl = (size_t)path_offsets_h[b0 + nb] - p0;
            cudaStream_t si = pipe->s_in;
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(S, b0 * slot_state), at(S_h, b0 * slot_state), nb * slot_state, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(q, n0 * row_qk), at(q_h, n0 * row_qk), nn * row_qk, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(k, n0 * row_qk), at(k_h, n0 * row_qk), nn * row_qk, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(v, n0 * row_v), at(v_h, n0 * row_v), nn * row_v, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(kp, m0 * row_qk), at(k_prev_h, m0 * row_qk), mm * row_qk, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaMemcpyAsync(atw(vp, m0 * row_v), at(v_prev_h, m0 * row_v), mm * row_v, cudaMemcpyHostToDevice, si));
            GDN_CUDA_TRY(cudaEventRecord(pipe->in[i], si));
            GDN_CUDA_TRY(cudaStreamWaitEvent(stream, pipe->in[i], 0));
            gdn_shape_t gs = s;
            gs.n_seq = nb;
            gs.total_nodes = (int32_t)nn;
            if (nn > 0 || pl > 0) {
                rc = gdn_tree_commit_verify(&gs, S + (size_t)b0 * (slot_state / sizeof(float)), at(kp, m0 * row_qk),
                                            at(vp, m0 * row_v), at(gp, m0 * row_gb), at(bp, m0 * row_gb),
                                            parent_p ? parent_p + m0 : nullptr, g_offs_p + b0 + i, path + p0,
                                            g_poffs + b0 + i, at(q, n0 * row_qk), at(k, n0 * row_qk), at(v, n0 * row_v),
                                            at(g, n0 * row_gb), at(beta, n0 * row_gb), parent + n0, g_offs + b0 + i,
                                            atw(o, n0 * row_o), ws, lay.total, status, cuda_stream);
                if (rc != GDN_OK) {   // refused on the host: let what is in flight drain before returning
                    cudaStreamSynchronize(pipe->s_in);
                    cudaStreamSynchronize(stream);
                    cudaStreamSynchronize(pipe->s_out);
                    return rc;
                }
            }
            GDN_CUDA_TRY(cudaEventRecord(pipe->k[i], stream));
            cudaStream_t so = pipe->s_out;
            GDN_CUDA_TRY(cudaStreamWaitEvent(so, pipe->k[i], 0));
            if (nn) GDN_CUDA_TRY(cudaMemcpyAsync(atw(o_h, n0 * row_o), at(o, n0 * row_o), nn * row_o, cudaMemcpyDeviceToHost, so));
            if (pl) GDN_CUDA_TRY(cudaMemcpyAsync(atw(S_h, b0 * slot_state), at(S, b0 * slot_state), nb * slot_state, cudaMemcpyDeviceToHost, so));
        }
        GDN_CUDA_TRY(cudaEventRecord(pipe->done, pipe->s_out));
        GDN_CUDA_TRY(cudaStreamWaitEvent(stream, pipe->done, 0));
        int32_t status_p = 0;
        GDN_CUDA_TRY(cudaMemcpyAsync(&status_p, status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        GDN_CUDA_TRY(cudaStreamSynchronize(stream));
        return status_p;
    }
    // one copy of the state for both halves of the step: it goes up once and comes back once
    GDN_CUDA_TRY(cudaMemcpyAsync(S, S_h, t.state, cudaMemcpyHostToDevice, stream));
    if (total_path_len > 0) {
        GDN_CUDA_TRY(cudaMemcpyAsync(kp, k_prev_h, tp.qk, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(vp, v_prev_h, tp.v, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(gp, g_prev_h, tp.gb, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(bp, beta_prev_h, tp.gb, cudaMemcpyHostToDevice, stream));
        if (parent_p) GDN_CUDA_TRY(cudaMemcpyAsync(parent_p, parent_prev_h, tp.parent, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(path, path_h, path_bytes, cudaMemcpyHostToDevice, stream));
    }
    GDN_CUDA_TRY(cudaMemcpyAsync(offs_p, node_offsets_prev_h, tp.offsets, cudaMemcpyHostToDevice, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(poffs, path_offsets_h, tp.offsets, cudaMemcpyHostToDevice, stream));
    if (s.total_nodes > 0) {
        GDN_CUDA_TRY(cudaMemcpyAsync(q, q_h, t.qk, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(k, k_h, t.qk, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(v, v_h, t.v, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(g, g_h, t.gb, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(beta, beta_h, t.gb, cudaMemcpyHostToDevice, stream));
        GDN_CUDA_TRY(cudaMemcpyAsync(parent, parent_h, t.parent, cudaMemcpyHostToDevice, stream));
    }
    GDN_CUDA_TRY(cudaMemcpyAsync(offs, node_offsets_h, t.offsets, cudaMemcpyHostToDevice, stream));
    if (total_path_len > 0 || s.total_nodes > 0) {
        rc = gdn_tree_commit_verify(shape, S, kp, vp, gp, bp, parent_p, offs_p, path, poffs, q, k, v, g, beta, parent,
                                    offs, o, ws, lay.total, status, cuda_stream);
        if (rc != GDN_OK) return rc;
    }
    int32_t status_h = 0;
    if (s.total_nodes > 0) GDN_CUDA_TRY(cudaMemcpyAsync(o_h, o, t.o, cudaMemcpyDeviceToHost, stream));
    if (total_path_len > 0) GDN_CUDA_TRY(cudaMemcpyAsync(S_h, S, t.state, cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaMemcpyAsync(&status_h, status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    GDN_CUDA_TRY(cudaStreamSynchronize(stream));
    return status_h;
}
