// Commit kernel: replay Eq. 7 along the accepted root path and write the state in place
// (Section 3.4: the commit is delayed until the accepted branch is known and is "a short
// recurrence"; Section 3.4.2: it is the only state write of a decode step).
//
// With S' = alpha S (decay first), Eq. 7 reads S <- S' - beta k (k^T S') + beta k v^T, i.e. per
// value component c (one contiguous row of the [d_v][d_k] tile):
//     s_c <- alpha s_c + k * beta (v_c - alpha (k . s_c)).
// One CTA per (tree, value head); thread (c, s) owns 32 floats of row c (quarter s of the key
// dimension, interleaved in 16-byte pieces so that the four lanes of a row read 64 contiguous
// bytes) and k . s_c is reduced over the four lanes with warp shuffles.  The path nodes' k rows
// are fetched once into shared memory; the state is read once and written once.  The state loads
// are issued before anything else so that the path checks and the k-row staging run under their
// latency, and the kernel keeps to 64 registers so that two CTAs (32 warps) share an SM.
#include "gdn_internal.cuh"
#include "gdn_plan.cuh"
#include "gdn_replay.cuh"

namespace gdn {

namespace {

constexpr int CM_THREADS = 512;
constexpr int CM_SPLIT = 4;
constexpr int CM_DK = GDN_MAX_HEAD_DIM;
constexpr int CM_REGS = CM_DK / CM_SPLIT;

struct CommitParams {
    int h_qk, h_v, d_k, d_v, max_depth;
    float *S;
    const void *k, *v, *g, *beta;
    const int32_t *parent, *node_offsets, *path, *path_offsets;
    int32_t *status_dev;
    // padded layout (tile kernel only; t_pad = 0: ragged packing): slot b keeps its rows at b * t_pad and carries
    // tree b % n_trees, whose parent[] row, node count and accepted path are shared by its slots
    int t_pad, n_trees, path_stride, raw_gates;
    const int32_t *n_nodes, *path_len;
};

template <typename TIn>
__global__ void __launch_bounds__(CM_THREADS, 2) commit_generic_kernel(const CommitParams p)
{
    extern __shared__ __align__(16) float cm_smem[];
    float (*ks)[CM_DK] = reinterpret_cast<float (*)[CM_DK]>(cm_smem);   // [L][CM_DK]
    float *alpha_s = cm_smem + (size_t)p.max_depth * CM_DK;             // [L]
    float *beta_s = alpha_s + p.max_depth;                              // [L]
    int *path_s = reinterpret_cast<int *>(beta_s + p.max_depth);        // [L] node ids
    int *par_s = path_s + p.max_depth;                                  // [L] their parents
    __shared__ int path_bad;

    const int b = blockIdx.x / p.h_v, h = blockIdx.x % p.h_v;
    const int p0 = p.path_offsets[b];
    const int L = p.path_offsets[b + 1] - p0;
    if (L == 0) return;   // nothing accepted from this tree: state untouched
    const int base = p.node_offsets[b];
    const int T = p.node_offsets[b + 1] - base;
    const int tid = threadIdx.x;
    const int d_k = p.d_k, d_v = p.d_v;
    const bool shape_ok = L > 0 && L <= p.max_depth && T > 0 && p0 >= 0;

    const int hk = h / (p.h_v / p.h_qk);
    const int c = tid / CM_SPLIT, s = tid % CM_SPLIT;
    const bool comp_on = c < d_v;
    const TIn *k = static_cast<const TIn *>(p.k), *v = static_cast<const TIn *>(p.v);
    const TIn *g = static_cast<const TIn *>(p.g), *beta = static_cast<const TIn *>(p.beta);

    // The state slice goes first: its latency covers the path checks and the k-row staging below.
    float *row = p.S + ((size_t)(b * p.h_v + h) * d_v + (comp_on ? c : 0)) * d_k;
    float sreg[CM_REGS];
#pragma unroll
    for (int j = 0; j < CM_REGS / 4; ++j) {
        const int r = 16 * j + 4 * s;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (shape_ok && comp_on && r < d_k) x = *reinterpret_cast<const float4 *>(row + r);
        sreg[4 * j + 0] = x.x; sreg[4 * j + 1] = x.y; sreg[4 * j + 2] = x.z; sreg[4 * j + 3] = x.w;
    }

    // The accepted path must be a chain from a root inside this tree: every thread t < L fetches
    // its entry (and that node's parent) in parallel, thread 0 then checks the chain.
    if (shape_ok && tid < L) {
        const int n = p.path[p0 + tid];
        path_s[tid] = n;
        par_s[tid] = (p.parent && n >= 0 && n < T) ? p.parent[base + n] : -2;
    }
    __syncthreads();
    if (tid == 0) {
        int bad = !shape_ok;
        for (int t = 0; !bad && t < L; ++t) {
            const int n = path_s[t];
            if (n < 0 || n >= T) bad = 1;
            else if (p.parent) bad = par_s[t] != (t ? path_s[t - 1] : -1);
            else if (t && n <= path_s[t - 1]) bad = 1;   // without parent[] only the topological order can be checked
        }
        path_bad = bad;
        if (bad) report_status(p.status_dev, GDN_ERR_PATH);
    }
    __syncthreads();
    if (path_bad) return;

    // k rows of the path (fp32, zero padded to CM_DK) and the per-step scalars
    for (int idx = tid; idx < L * CM_DK; idx += CM_THREADS) {
        const int t = idx / CM_DK, r = idx % CM_DK;
        const size_t n = (size_t)base + path_s[t];
        ks[t][r] = r < d_k ? load_as_float(k + (n * p.h_qk + hk) * d_k + r) : 0.f;
    }
    if (tid < L) {
        const size_t n = (size_t)base + path_s[tid];
        alpha_s[tid] = expf(load_as_float(g + n * p.h_v + h));
        beta_s[tid] = load_as_float(beta + n * p.h_v + h);
    }
    float vc = comp_on ? load_as_float(v + (((size_t)base + path_s[0]) * p.h_v + h) * d_v + c) : 0.f;
    __syncthreads();

    for (int t = 0; t < L; ++t) {
        float vnext = 0.f;   // next step's v[c], fetched while this step computes
        if (comp_on && t + 1 < L)
            vnext = load_as_float(v + (((size_t)base + path_s[t + 1]) * p.h_v + h) * d_v + c);
        float dot = 0.f;
#pragma unroll
        for (int j = 0; j < CM_REGS / 4; ++j) {
            const float4 kx = *reinterpret_cast<const float4 *>(&ks[t][16 * j + 4 * s]);
            dot = fmaf(kx.x, sreg[4 * j + 0], dot); dot = fmaf(kx.y, sreg[4 * j + 1], dot);
            dot = fmaf(kx.z, sreg[4 * j + 2], dot); dot = fmaf(kx.w, sreg[4 * j + 3], dot);
        }
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
        dot += __shfl_xor_sync(0xffffffffu, dot, 2);
        const float alpha = alpha_s[t];
        const float w = beta_s[t] * (vc - alpha * dot);
#pragma unroll
        for (int j = 0; j < CM_REGS / 4; ++j) {
            const float4 kx = *reinterpret_cast<const float4 *>(&ks[t][16 * j + 4 * s]);
            sreg[4 * j + 0] = fmaf(kx.x, w, alpha * sreg[4 * j + 0]);
            sreg[4 * j + 1] = fmaf(kx.y, w, alpha * sreg[4 * j + 1]);
            sreg[4 * j + 2] = fmaf(kx.z, w, alpha * sreg[4 * j + 2]);
            sreg[4 * j + 3] = fmaf(kx.w, w, alpha * sreg[4 * j + 3]);
        }
        vc = vnext;
    }

    if (comp_on) {
#pragma unroll
        for (int j = 0; j < CM_REGS / 4; ++j) {
            const int r = 16 * j + 4 * s;
            if (r < d_k)
                *reinterpret_cast<float4 *>(row + r) =
                    make_float4(sreg[4 * j + 0], sreg[4 * j + 1], sreg[4 * j + 2], sreg[4 * j + 3]);
        }
    }
}

// Fast form for d_k = d_v = 128, bf16 inputs, paths of at most 16 nodes: 256 threads hold the tile as the
// tensor-core verify kernel does (eight lanes per row, 32-byte accesses) and replay the path in the scaled form
// (gdn_replay.cuh).  One CTA per (tree, value head), two CTAs per SM; the state loads go first, the path is fetched
// and checked by one warp with shuffles, its k/v rows arrive by cp.async.
constexpr int CF_THREADS = 256;
constexpr int CF_MD = 16;

__device__ __forceinline__ void cf_cp_async_16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__device__ __forceinline__ void commit_tile128_unit(const CommitParams &p, const int unit)
{
    __shared__ __align__(16) uint16_t pk_s[CF_MD * GDN_TILE_D];
    __shared__ __align__(16) uint16_t pv_s[CF_MD * GDN_TILE_D];
    __shared__ __align__(16) float4 ab_s[CF_MD];
    __shared__ int len_s;

    const int b = unit / p.h_v, h = unit % p.h_v;
    const int hk = h / (p.h_v / p.h_qk);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r4 = lane >> 3, l8 = lane & 7;
    const int tree = p.t_pad ? b % p.n_trees : b;
    const int pp0 = p.t_pad ? tree * p.path_stride : p.path_offsets[b];
    int len = p.t_pad ? p.path_len[tree] : p.path_offsets[b + 1] - pp0;
    if (len == 0) return;   // nothing accepted from this tree: state untouched

    // the state tile first: its latency covers the path fetch below
    float *S = p.S + (size_t)(b * p.h_v + h) * GDN_TILE_D * GDN_TILE_D;
    float4 x[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float *src = S + (size_t)(warp * 16 + i * 4 + r4) * GDN_TILE_D + l8 * 8;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) ldg_v8(src + kh * 64, x[i][kh * 2 + 0], x[i][kh * 2 + 1]);
    }

    const int pb = p.t_pad ? b * p.t_pad : p.node_offsets[b];
    const int pT = p.t_pad ? min(p.n_nodes[tree], p.t_pad) : p.node_offsets[b + 1] - pb;
    const int ppar = p.t_pad ? tree * p.t_pad : pb;   // first entry of the tree in parent[]
    const __nv_bfloat16 *k = static_cast<const __nv_bfloat16 *>(p.k), *v = static_cast<const __nv_bfloat16 *>(p.v);
    const __nv_bfloat16 *g = static_cast<const __nv_bfloat16 *>(p.g), *beta = static_cast<const __nv_bfloat16 *>(p.beta);
    const bool shape_ok = len > 0 && len <= CF_MD && len <= p.max_depth && pT > 0 && pp0 >= 0;
    // Every thread reads the path entry whose row piece it fetches (no hand-over through shared memory in front of
    // the row fetch); an entry outside the tree is skipped here and reported by the check below.
    if (shape_ok) {
        for (int idx = tid; idx < len * 32; idx += CF_THREADS) {
            const int t = idx >> 5, c16 = idx & 15;
            const int nt = p.path[pp0 + t];
            if (nt < 0 || nt >= pT) continue;
            const size_t n = (size_t)pb + nt;
            if (idx & 16)
                cf_cp_async_16((uint32_t)__cvta_generic_to_shared(pv_s + t * GDN_TILE_D + c16 * 8),
                               v + (n * p.h_v + h) * GDN_TILE_D + c16 * 8);
            else
                cf_cp_async_16((uint32_t)__cvta_generic_to_shared(pk_s + t * GDN_TILE_D + c16 * 8),
                               k + (n * p.h_qk + hk) * GDN_TILE_D + c16 * 8);
        }
    }
    if (warp == 0) {
        // lane t: entry t of the path and that node's parent; the path must be a chain from a root inside the tree
        const bool mine = shape_ok && lane < len;
        int n = -1, parent_n = -2;
        if (mine) {
            n = p.path[pp0 + lane];
            if (p.parent && n >= 0 && n < pT) parent_n = p.parent[ppar + n];
        }
        const int n_up = __shfl_up_sync(0xffffffffu, n, 1);
        bool bad = false;
        if (mine) {
            if (n < 0 || n >= pT) bad = true;
            else if (p.parent) bad = parent_n != (lane ? n_up : -1);
            else if (lane && n <= n_up) bad = true;   // without parent[] only the topological order can be checked
        }
        if (__any_sync(0xffffffffu, bad) || !shape_ok) {
            if (lane == 0) report_status(p.status_dev, GDN_ERR_PATH);
            len = 0;
        }
        // per-step scalars: decay of the path up to and including step t by a prefix sum over the lanes
        float gt = 0.f, be = 0.f;
        if (lane < len) {
            const unsigned short *g16 = reinterpret_cast<const unsigned short *>(g);
            const unsigned short *b16 = reinterpret_cast<const unsigned short *>(beta);
            gt = gate_log_decay(g16[((size_t)pb + n) * p.h_v + h], p.raw_gates != 0);
            be = gate_beta(b16[((size_t)pb + n) * p.h_v + h], p.raw_gates != 0);
        }
        float gsum = gt;
#pragma unroll
        for (int off = 1; off < CF_MD; off <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, gsum, off);
            if (lane >= off) gsum += up;
        }
        if (lane < len) {
            const float A = expf(gsum);
            ab_s[lane] = make_float4(A, be, expf(gt), 1.f / A);
        }
        if (lane == 0) len_s = len;
    }
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    len = len_s;
    if (len == 0) return;   // rejected path: this state stays as it was

    replay_path_on_tile(x, len, pk_s, pv_s, ab_s, warp, r4, l8);

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float *dst = S + (size_t)(warp * 16 + i * 4 + r4) * GDN_TILE_D + l8 * 8;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) stg_v8(dst + kh * 64, x[i][kh * 2 + 0], x[i][kh * 2 + 1]);
    }
}

__global__ void __launch_bounds__(CF_THREADS, 2) commit_tile128_kernel(const CommitParams p)
{
    commit_tile128_unit(p, (int)blockIdx.x);
}

// The fused call on trees of more than 64 nodes: the plans of the NEW trees do not depend on the commit of the previous
// step's paths, so they are built by the first n_seq CTAs of the same grid instead of by a launch of their own in
// between (one launch and one dependency hop less in front of the verify kernel).
static_assert(PLAN_THREADS == CF_THREADS, "the plan CTAs and the commit CTAs share a block size");
__global__ void __launch_bounds__(CF_THREADS, 2) commit_plan_kernel(const CommitParams p, const PlanArgs a)
{
    if ((int)blockIdx.x < a.n_seq)
        plan_tree(a, (int)blockIdx.x);
    else
        commit_tile128_unit(p, (int)blockIdx.x - a.n_seq);
}

}  // namespace

cudaError_t launch_commit_generic(const gdn_shape_t &s, float *S, const void *k, const void *v,
                                  const void *g, const void *beta, const int32_t *parent,
                                  const int32_t *node_offsets, const int32_t *path,
                                  const int32_t *path_offsets, int32_t *status_dev, cudaStream_t stream)
{
    const int grid = s.n_seq * s.h_v;
    if (grid == 0) return cudaSuccess;
    CommitParams p{s.h_qk, s.h_v, s.d_k, s.d_v, s.max_depth, S, k, v, g, beta,
                   parent, node_offsets, path, path_offsets, status_dev, 0, 0, 0, 0, nullptr, nullptr};
    if (s.d_k == GDN_TILE_D && s.d_v == GDN_TILE_D && s.in_dtype == GDN_BF16 && s.max_depth <= CF_MD) {
        commit_tile128_kernel<<<grid, CF_THREADS, 0, stream>>>(p);
        return cudaGetLastError();
    }
    const size_t smem = sizeof(float) * ((size_t)s.max_depth * CM_DK + 4 * (size_t)s.max_depth);
    cudaError_t e;
    if (s.in_dtype == GDN_BF16) {
        e = cudaFuncSetAttribute(commit_generic_kernel<__nv_bfloat16>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        commit_generic_kernel<__nv_bfloat16><<<grid, CM_THREADS, smem, stream>>>(p);
    } else {
        e = cudaFuncSetAttribute(commit_generic_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        commit_generic_kernel<float><<<grid, CM_THREADS, smem, stream>>>(p);
    }
    return cudaGetLastError();
}

bool commit_tile128_supported(const gdn_shape_t &s) { return commit_padded_supported(s); }

// Commit of the previous step's paths (ragged packing, tile kernel) and the plan of the new trees in one grid.
cudaError_t launch_commit_plan(const gdn_shape_t &s, float *S, const void *k, const void *v, const void *g,
                               const void *beta, const int32_t *parent_prev, const int32_t *node_offsets_prev,
                               const int32_t *path, const int32_t *path_offsets, const int32_t *parent,
                               const int32_t *node_offsets, const PlanPtrs &plan, int32_t *status_dev,
                               cudaStream_t stream)
{
    if (s.n_seq == 0) return cudaSuccess;
    if (s.n_seq > 1) {   // the trees' CTAs claim their places in the unit list from a counter
        cudaError_t e0 = cudaMemsetAsync(plan.unit_count, 0, sizeof(int32_t), stream);
        if (e0 != cudaSuccess) return e0;
    }
    CommitParams p{s.h_qk, s.h_v, s.d_k, s.d_v, s.max_depth, S, k, v, g, beta, parent_prev, node_offsets_prev, path,
                   path_offsets, status_dev, 0, 0, 0, 0, nullptr, nullptr};
    const int grid = s.n_seq + s.n_seq * s.h_v;
    commit_plan_kernel<<<grid, CF_THREADS, 0, stream>>>(p, plan_args(s, parent, node_offsets, nullptr, plan, status_dev));
    return cudaGetLastError();
}

bool commit_padded_supported(const gdn_shape_t &s)
{
    return s.d_k == GDN_TILE_D && s.d_v == GDN_TILE_D && s.in_dtype == GDN_BF16 && s.max_depth <= CF_MD;
}

cudaError_t launch_commit_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, float *S, const void *k,
                                 const void *v, const void *g, const void *beta, const int32_t *parent,
                                 const int32_t *n_nodes, const int32_t *path, const int32_t *path_len,
                                 int32_t *status_dev, cudaStream_t stream)
{
    const int grid = s.n_seq * s.h_v;
    if (grid == 0) return cudaSuccess;
    CommitParams p{s.h_qk, s.h_v, s.d_k, s.d_v, s.max_depth, S, k, v, g, beta, parent, nullptr, path, nullptr,
                   status_dev, s.max_tree_nodes, n_trees, s.max_depth, raw_gates ? 1 : 0, n_nodes, path_len};
    commit_tile128_kernel<<<grid, CF_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace gdn
