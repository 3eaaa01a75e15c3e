// Generic tree-verify kernel: any d_k, d_v <= 128, fp32 or bf16 inputs, CUDA cores only.
//
// It evaluates the triangular form of Section 3.4.1 restricted to real ancestors.  With
// dec(i,j) = exp(sum of g over the nodes after j up to and including i on i's root path)
// (= a_i / a_j of Eq. 9, formed as a suffix sum so that no large exponents cancel):
//     p^k_i = S0^T k_i,  p^q_i = S0^T q_i                          (the S0 terms of Eq. 11 / 13)
//     u~_i  = beta_i (v_i - a_i p^k_i) - sum_{j < i on path} dec(i,j) beta_i (k_i.k_j) u~_j   (Eq. 10, 13)
//     o_i   = scale (a_i p^q_i + sum_{j <= i on path} dec(i,j) (q_i.k_j) u~_j)              (Eq. 11)
// u~_i = u_i - w_i^T S0 is the quantity the substitution returns once the W S0 term is folded
// into the right-hand side (Section 3.4.2), so W is never formed.
//
// One CTA per (tree, value head).  Thread (c, s): value component c, quarter s of the key
// dimension; the [d_v][d_k] state tile lives in registers (32 floats per thread) and the two
// projections are reduced over the four s-lanes with warp shuffles.  Nodes are visited in index
// order (parents first); u~ is kept in the workspace (L2) because a tree may be larger than
// shared memory allows.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int VG_THREADS = 512;
constexpr int VG_SPLIT = 4;                      // lanes sharing one value component
constexpr int VG_CHUNK = 32;                     // nodes whose coefficients are prepared together
constexpr int VG_DK = GDN_MAX_HEAD_DIM;          // padded key dim in shared memory
constexpr int VG_REGS = VG_DK / VG_SPLIT;        // state floats per thread
constexpr int VG_WARPS = VG_THREADS / 32;

struct VerifyGenericParams {
    int h_qk, h_v, d_k, d_v, max_depth;
    float scale;
    const float *S0;
    const void *q, *k, *v, *g, *beta;
    const int32_t *node_offsets;
    void *o;
    const int32_t *tree_ok;
    const uint8_t *depth;
    const uint16_t *anc;
    float *utilde;
};

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(VG_THREADS, 1) verify_generic_kernel(const VerifyGenericParams p)
{
    extern __shared__ __align__(16) float vg_smem[];
    float (*ks)[VG_DK] = reinterpret_cast<float (*)[VG_DK]>(vg_smem);
    float (*qs)[VG_DK] = ks + VG_CHUNK;
    float *xc = &qs[VG_CHUNK][0];                 // [VG_CHUNK][max_depth]: dec, then X coefficients
    float *yc = xc + VG_CHUNK * p.max_depth;      // [VG_CHUNK][max_depth]: Y coefficients (self included)
    float *a_s = yc + VG_CHUNK * p.max_depth;     // [VG_CHUNK]
    float *beta_s = a_s + VG_CHUNK;               // [VG_CHUNK]

    const int b = blockIdx.x / p.h_v, h = blockIdx.x % p.h_v;
    if (!p.tree_ok[b]) return;
    const int base = p.node_offsets[b];
    const int T = p.node_offsets[b + 1] - base;
    if (T <= 0) return;
    const int hk = h / (p.h_v / p.h_qk);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = tid / VG_SPLIT, s = tid % VG_SPLIT;
    const bool comp_on = c < p.d_v;
    const int d_k = p.d_k, d_v = p.d_v, md = p.max_depth;

    const TIn *q = static_cast<const TIn *>(p.q), *k = static_cast<const TIn *>(p.k);
    const TIn *v = static_cast<const TIn *>(p.v), *g = static_cast<const TIn *>(p.g);
    const TIn *beta = static_cast<const TIn *>(p.beta);
    TOut *o = static_cast<TOut *>(p.o);

    // State slice: register 4*j+e holds S0[c][16*j + 4*s + e] (zero beyond d_k / d_v).
    float sreg[VG_REGS];
    {
        const float *row = p.S0 + ((size_t)(b * p.h_v + h) * d_v + (comp_on ? c : 0)) * d_k;
#pragma unroll
        for (int j = 0; j < VG_REGS / 4; ++j) {
            const int r = 16 * j + 4 * s;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (comp_on && r < d_k) x = __ldg(reinterpret_cast<const float4 *>(row + r));
            sreg[4 * j + 0] = x.x; sreg[4 * j + 1] = x.y; sreg[4 * j + 2] = x.z; sreg[4 * j + 3] = x.w;
        }
    }
    for (int idx = tid; idx < VG_CHUNK * VG_DK; idx += VG_THREADS) {
        (&ks[0][0])[idx] = 0.f;
        (&qs[0][0])[idx] = 0.f;
    }

    for (int i0 = 0; i0 < T; i0 += VG_CHUNK) {
        const int cn = min(VG_CHUNK, T - i0);
        __syncthreads();   // previous chunk fully consumed (and the zero fill done)
        // (a) stage this chunk's k and q rows as fp32
        for (int idx = tid; idx < cn * d_k; idx += VG_THREADS) {
            const int t = idx / d_k, r = idx % d_k;
            const size_t src = ((size_t)(base + i0 + t) * p.h_qk + hk) * d_k + r;
            ks[t][r] = load_as_float(k + src);
            qs[t][r] = load_as_float(q + src);
        }
        // (b0) per node: decay from each path position to the node, total decay a_i, beta_i
        if (tid < cn) {
            const int n = base + i0 + tid;
            const int d = p.depth[n];
            const uint16_t *path = p.anc + (size_t)n * md;
            float sfx = 0.f;
            for (int a = d - 1; a >= 0; --a) {
                xc[tid * md + a] = expf(sfx);
                sfx += load_as_float(g + (size_t)(base + path[a]) * p.h_v + h);
            }
            a_s[tid] = expf(sfx);
            beta_s[tid] = load_as_float(beta + (size_t)n * p.h_v + h);
        }
        __syncthreads();
        // (b) one warp per (node, path position): k_i.k_j and q_i.k_j, scaled into X and Y of Eq. 9
        for (int idx = warp; idx < cn * md; idx += VG_WARPS) {
            const int t = idx / md, a = idx % md;
            const int n = base + i0 + t;
            const int d = p.depth[n];
            if (a >= d) continue;
            const int j = p.anc[(size_t)n * md + a];
            const TIn *kj = k + ((size_t)(base + j) * p.h_qk + hk) * d_k;
            float kk = 0.f, qk = 0.f;
            for (int r = lane; r < d_k; r += 32) {
                const float x = load_as_float(kj + r);
                kk = fmaf(ks[t][r], x, kk);
                qk = fmaf(qs[t][r], x, qk);
            }
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                kk += __shfl_xor_sync(0xffffffffu, kk, m);
                qk += __shfl_xor_sync(0xffffffffu, qk, m);
            }
            if (lane == 0) {
                const float dec = xc[t * md + a];
                yc[t * md + a] = dec * qk;
                xc[t * md + a] = beta_s[t] * dec * kk;   // entry a = d-1 (the node itself) is never read
            }
        }
        __syncthreads();
        // (c) nodes in order: projections, forward substitution step, output
        for (int t = 0; t < cn; ++t) {
            const int n = base + i0 + t;
            float pk = 0.f, pq = 0.f;
#pragma unroll
            for (int j = 0; j < VG_REGS / 4; ++j) {
                const float4 kx = *reinterpret_cast<const float4 *>(&ks[t][16 * j + 4 * s]);
                const float4 qx = *reinterpret_cast<const float4 *>(&qs[t][16 * j + 4 * s]);
                pk = fmaf(sreg[4 * j + 0], kx.x, pk); pk = fmaf(sreg[4 * j + 1], kx.y, pk);
                pk = fmaf(sreg[4 * j + 2], kx.z, pk); pk = fmaf(sreg[4 * j + 3], kx.w, pk);
                pq = fmaf(sreg[4 * j + 0], qx.x, pq); pq = fmaf(sreg[4 * j + 1], qx.y, pq);
                pq = fmaf(sreg[4 * j + 2], qx.z, pq); pq = fmaf(sreg[4 * j + 3], qx.w, pq);
            }
            pk += __shfl_xor_sync(0xffffffffu, pk, 1); pk += __shfl_xor_sync(0xffffffffu, pk, 2);
            pq += __shfl_xor_sync(0xffffffffu, pq, 1); pq += __shfl_xor_sync(0xffffffffu, pq, 2);

            const int d = p.depth[n];
            const uint16_t *path = p.anc + (size_t)n * md;
            float sx = 0.f, sy = 0.f;   // partial sums over this lane's share of the ancestors
            if (comp_on) {
                for (int a = s; a < d - 1; a += VG_SPLIT) {
                    const float uj = __ldcg(p.utilde + ((size_t)(base + path[a]) * p.h_v + h) * d_v + c);
                    sx = fmaf(xc[t * md + a], uj, sx);
                    sy = fmaf(yc[t * md + a], uj, sy);
                }
            }
            sx += __shfl_xor_sync(0xffffffffu, sx, 1); sx += __shfl_xor_sync(0xffffffffu, sx, 2);
            sy += __shfl_xor_sync(0xffffffffu, sy, 1); sy += __shfl_xor_sync(0xffffffffu, sy, 2);
            if (comp_on) {
                const float vi = load_as_float(v + ((size_t)n * p.h_v + h) * d_v + c);
                const float ui = beta_s[t] * (vi - a_s[t] * pk) - sx;
                const float out = p.scale * (fmaf(a_s[t], pq, sy) + yc[t * md + d - 1] * ui);
                if (s == 0) {
                    __stcg(p.utilde + ((size_t)n * p.h_v + h) * d_v + c, ui);
                    store_from_float(o + ((size_t)n * p.h_v + h) * d_v + c, out);
                }
            }
            __syncwarp();   // lane s==0's u~ store is ordered before the other lanes' later loads
        }
    }
}

template <typename TIn, typename TOut>
cudaError_t launch_typed(const gdn_shape_t &s, const VerifyGenericParams &p, cudaStream_t stream)
{
    const int grid = s.n_seq * s.h_v;
    if (grid == 0 || s.total_nodes == 0) return cudaSuccess;
    const size_t smem = sizeof(float) * (2 * VG_CHUNK * VG_DK + 2 * VG_CHUNK * (size_t)s.max_depth + 2 * VG_CHUNK);
    cudaError_t e = cudaFuncSetAttribute(verify_generic_kernel<TIn, TOut>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    verify_generic_kernel<TIn, TOut><<<grid, VG_THREADS, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_verify_generic(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                  const void *v, const void *g, const void *beta,
                                  const int32_t *node_offsets, void *o, const PlanPtrs &plan,
                                  cudaStream_t stream)
{
    VerifyGenericParams p{s.h_qk, s.h_v, s.d_k, s.d_v, s.max_depth, s.scale, S0, q, k, v, g, beta,
                          node_offsets, o, plan.tree_ok, plan.depth, plan.anc, plan.utilde};
    const bool in_bf = s.in_dtype == GDN_BF16, out_bf = s.out_dtype == GDN_BF16;
    if (in_bf && out_bf) return launch_typed<__nv_bfloat16, __nv_bfloat16>(s, p, stream);
    if (in_bf) return launch_typed<__nv_bfloat16, float>(s, p, stream);
    if (out_bf) return launch_typed<float, __nv_bfloat16>(s, p, stream);
    return launch_typed<float, float>(s, p, stream);
}

}  // namespace gdn
