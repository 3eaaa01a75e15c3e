// Per-branch recurrent tree verification: the baseline that Section 3.4 sets the rollback-free kernel against
// ("sequential scans along tree branches") and that Section 5.2 / Figure 5 times next to the fused kernel.
//
// One CTA per (tree, value head, leaf).  It copies the state tile S0 of its head into registers and runs Eq. 7
// token by token down the root path of its leaf, writing o_i = scale q_i^T S_i (Eq. 8) for every node i it passes.
// Branches that share a prefix recompute it (no parent-state reuse): every branch writes the outputs of its whole
// path, and since each branch performs the same operations in the same order on a shared node, concurrent writers
// store identical bits.  S0 is never written.  This kernel exists as a comparator and as a second, structurally
// different check of the tensor-core path; it is not tuned.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int VR_THREADS = 256;   // thread (c, s): value component c = tid / 2, half s of the key dimension
constexpr int VR_HALF = GDN_MAX_HEAD_DIM / 2;

struct VerifyRecurrentParams {
    int h_qk, h_v, d_k, d_v, max_depth, max_tree_nodes, total_nodes, n_seq;
    float scale;
    const float *S0;
    const void *q, *k, *v, *g, *beta;
    const int32_t *parent, *node_offsets;
    void *o;
    int32_t *status_dev;
};

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(VR_THREADS) verify_recurrent_kernel(const VerifyRecurrentParams p)
{
    __shared__ int path_s[GDN_MAX_DEPTH_CAP];
    __shared__ float kq_s[2][GDN_MAX_HEAD_DIM];   // k row and q row of the current node
    __shared__ int has_child, path_len_s, err_s;

    const int b = blockIdx.x / p.h_v, h = blockIdx.x % p.h_v;
    const int leaf = blockIdx.y;
    const int base = p.node_offsets[b];
    const int T = p.node_offsets[b + 1] - base;
    if (base < 0 || T <= 0 || T > p.max_tree_nodes || base + T > p.total_nodes) {
        if (T != 0 && threadIdx.x == 0 && leaf == 0) report_status(p.status_dev, GDN_ERR_TREE);
        return;
    }
    if (leaf >= T) return;
    const int tid = threadIdx.x;
    if (tid == 0) {
        has_child = 0;
        err_s = 0;
    }
    __syncthreads();
    // a node is a leaf if no later node names it as its parent
    for (int j = leaf + 1 + tid; j < T; j += VR_THREADS)
        if (p.parent[base + j] == leaf) has_child = 1;
    __syncthreads();
    if (has_child) return;
    if (tid == 0) {   // root path of the leaf, leaf first; parent[] is checked on the way
        int d = 0, cur = leaf, err = 0;
        while (cur >= 0) {
            if (d >= p.max_depth) { err = GDN_ERR_DEPTH; break; }
            path_s[d++] = cur;
            const int par = p.parent[base + cur];
            if (par < -1 || par >= cur) { err = GDN_ERR_TREE; break; }
            cur = par;
        }
        if (err) report_status(p.status_dev, err);
        err_s = err;
        path_len_s = d;
    }
    __syncthreads();
    if (err_s) return;   // the ordinary verify rejects such a tree as a whole; here the faulty branch writes nothing
    const int L = path_len_s;

    const int c = tid >> 1, s = tid & 1;
    const int hk = h / (p.h_v / p.h_qk);
    const int d_k = p.d_k, d_v = p.d_v;
    const bool on = c < d_v;
    const TIn *q = static_cast<const TIn *>(p.q), *k = static_cast<const TIn *>(p.k);
    const TIn *v = static_cast<const TIn *>(p.v), *g = static_cast<const TIn *>(p.g);
    const TIn *beta = static_cast<const TIn *>(p.beta);
    TOut *o = static_cast<TOut *>(p.o);

    // state row c, key positions s*64 .. s*64+63 (zero beyond d_k)
    float st[VR_HALF];
    {
        const float *row = p.S0 + ((size_t)(b * p.h_v + h) * d_v + (on ? c : 0)) * d_k;
#pragma unroll
        for (int e = 0; e < VR_HALF; ++e) {
            const int r = s * VR_HALF + e;
            st[e] = (on && r < d_k) ? __ldg(row + r) : 0.f;
        }
    }
    for (int t = L - 1; t >= 0; --t) {   // root first
        const size_t n = (size_t)base + path_s[t];
        __syncthreads();
        if (tid < GDN_MAX_HEAD_DIM) kq_s[0][tid] = tid < d_k ? load_as_float(k + (n * p.h_qk + hk) * d_k + tid) : 0.f;
        else kq_s[1][tid - GDN_MAX_HEAD_DIM] =
                 tid - GDN_MAX_HEAD_DIM < d_k ? load_as_float(q + (n * p.h_qk + hk) * d_k + tid - GDN_MAX_HEAD_DIM) : 0.f;
        __syncthreads();
        const float alpha = expf(load_as_float(g + n * p.h_v + h));
        const float be = load_as_float(beta + n * p.h_v + h);
        const float vc = on ? load_as_float(v + (n * p.h_v + h) * d_v + c) : 0.f;
        // Eq. 7 for row c: s <- alpha (s - beta k (k.s)) + beta k v_c
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < VR_HALF; ++e) dot = fmaf(kq_s[0][s * VR_HALF + e], st[e], dot);
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
        const float w = be * (vc - alpha * dot);
        float oq = 0.f;
#pragma unroll
        for (int e = 0; e < VR_HALF; ++e) {
            st[e] = fmaf(kq_s[0][s * VR_HALF + e], w, alpha * st[e]);
            oq = fmaf(kq_s[1][s * VR_HALF + e], st[e], oq);
        }
        oq += __shfl_xor_sync(0xffffffffu, oq, 1);   // Eq. 8
        if (on && s == 0) store_from_float(o + (n * p.h_v + h) * d_v + c, p.scale * oq);
    }
}

template <typename TIn, typename TOut>
cudaError_t launch_typed(const gdn_shape_t &s, const VerifyRecurrentParams &p, cudaStream_t stream)
{
    const dim3 grid((unsigned)(s.n_seq * s.h_v), (unsigned)s.max_tree_nodes);
    verify_recurrent_kernel<TIn, TOut><<<grid, VR_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_verify_recurrent(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                    const void *v, const void *g, const void *beta, const int32_t *parent,
                                    const int32_t *node_offsets, void *o, int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyRecurrentParams p{};
    p.h_qk = s.h_qk; p.h_v = s.h_v; p.d_k = s.d_k; p.d_v = s.d_v; p.max_depth = s.max_depth;
    p.max_tree_nodes = s.max_tree_nodes; p.total_nodes = s.total_nodes; p.n_seq = s.n_seq; p.scale = s.scale;
    p.S0 = S0; p.q = q; p.k = k; p.v = v; p.g = g; p.beta = beta; p.parent = parent; p.node_offsets = node_offsets;
    p.o = o; p.status_dev = status_dev;
    const bool in_bf16 = s.in_dtype == GDN_BF16, out_bf16 = s.out_dtype == GDN_BF16;
    if (in_bf16) return out_bf16 ? launch_typed<__nv_bfloat16, __nv_bfloat16>(s, p, stream)
                                 : launch_typed<__nv_bfloat16, float>(s, p, stream);
    return out_bf16 ? launch_typed<float, __nv_bfloat16>(s, p, stream) : launch_typed<float, float>(s, p, stream);
}

}  // namespace gdn
