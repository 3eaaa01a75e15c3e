// Tree-verify fast path for sm_100a: d_k = d_v = 128, bf16 inputs, trees of at most 64 nodes,
// root paths of at most 16 nodes.  Same mathematics as the generic kernel (the triangular form of
// Section 3.4.1 restricted to real ancestors, W S0 folded into the right-hand side as in
// Section 3.4.2), but the dense part runs on the 5th-generation tensor cores:
//
//   P  [d_v x 2T] = S0 [d_v x d_k] . [K;Q]^T      (the S0 projections of Eq. 11 / Eq. 13: 86% of the FLOPs)
//   Gr [2T x T]   = [K;Q] . K^T                   (k_i.k_j and q_i.k_j of Eq. 9, per key head)
//
// Both are tcgen05.mma (kind::f16, bf16 operands, fp32 accumulators in tensor memory).  q and k
// are bf16 already; the fp32 state is split on the fly into two bf16 terms S0 = hi + lo
// (|S0 - hi - lo| <= 2^-16 |S0|), so P costs two accumulating MMA passes and keeps fp32-level
// accuracy.  Operand orientation: d_v on the TMEM lanes, nodes on the TMEM columns -- thread c of
// the first four warps then owns value component c of every node and runs the whole ancestor-
// masked substitution and the output for that component without exchanging data with any other
// thread (X and Y coefficients are broadcast from shared memory).
//
// One CTA per (tree, value head), 256 threads, about 108 KB of shared memory and 256 TMEM columns,
// so two CTAs share an SM: while one streams its 64 KB state tile from HBM the other computes.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int FV_THREADS = 256;
constexpr int FV_D = 128;           // d_k = d_v
constexpr int FV_T = 64;            // max nodes per tree
constexpr int FV_MD = 16;           // max nodes on a root path
constexpr int FV_TMEM_COLS = 256;   // P: columns [0,128), Gram: [128,192)
constexpr int FV_GRAM_PITCH = 65;   // floats per Gram row in shared memory (odd: conflict-free column writes)

// shared memory map (bytes from a 1024-byte aligned base)
constexpr int SM_A_HI = 0;                       // [2][128 rows][128 B], 128B-swizzled, K-major
constexpr int SM_A_LO = 32768;
constexpr int SM_B_KQ = 65536;                   // rows 0..63 = k of node r, rows 64..127 = q of node r-64
constexpr int SM_GRAM = 0;                       // after the MMAs: fp32 [128][65] over A_HI/A_LO
constexpr int SM_UT = SM_B_KQ;                   // after the MMAs: fp32 [64][128] over B_KQ
constexpr int SM_X = 98304;                      // fp32 [64][16]
constexpr int SM_Y = SM_X + FV_T * FV_MD * 4;    // fp32 [64][16]
constexpr int SM_A = SM_Y + FV_T * FV_MD * 4;    // fp32 [64] total decay a_i
constexpr int SM_BETA = SM_A + FV_T * 4;         // fp32 [64]
constexpr int SM_ANC = SM_BETA + FV_T * 4;       // u8 [64][16]
constexpr int SM_DEPTH = SM_ANC + FV_T * FV_MD;  // u8 [64]
constexpr int SM_MBAR = SM_DEPTH + FV_T;         // u64
constexpr int SM_TMEM = SM_MBAR + 8;             // u32
constexpr int SM_FLAG = SM_TMEM + 4;             // u32 (timeout flag)
constexpr int SM_BYTES = SM_FLAG + 4;
constexpr int SM_ALLOC = SM_BYTES + 1024;        // slack for the 1024-byte alignment of the base

struct VerifyFastParams {
    int h_qk, h_v, max_depth;   // max_depth = stride of the plan's ancestor table
    float scale;
    const float *S0;
    const __nv_bfloat16 *q, *k, *v, *g, *beta;
    const int32_t *node_offsets;
    void *o;
    const int32_t *tree_ok;
    const uint8_t *depth;
    const uint16_t *anc;
    int32_t *status_dev;
};

// ---------------------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 16 : 0;   // src-size 0: nothing is read, the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] . B[smem]^T, one K=16 step of a bf16 x bf16 -> fp32 MMA issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

#define GDN_TMEM_LD16(taddr, r)                                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, " \
                 "[%16];"                                                                                    \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),       \
                   "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),   \
                   "=r"(r[14]), "=r"(r[15])                                                                  \
                 : "r"(taddr)                                                                                \
                 : "memory")

// Shared-memory matrix descriptor: K-major, 128-byte swizzle (8-row groups of 1024 bytes).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) /* leading byte offset (unused when swizzled) */
           | (64ull << 32)                                  /* stride byte offset 1024 >> 4 */
           | (1ull << 46)                                   /* descriptor version of sm_100 */
           | (2ull << 61);                                  /* SWIZZLE_128B */
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// Byte offset of 16-byte piece `c16` (0..15 along K) of row `r` in a [2][128][128 B] swizzled tile.
__device__ __forceinline__ uint32_t sw128_offset(int r, int c16)
{
    return (uint32_t)((c16 >> 3) * 16384 + (r >> 3) * 1024 + (r & 7) * 128 + (((c16 & 7) ^ (r & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo_elem, float hi_elem)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo_elem, hi_elem);
    return *reinterpret_cast<uint32_t *>(&t);
}

// ---------------------------------------------------------------------------------------- kernel
template <typename TOut>
__global__ void __launch_bounds__(FV_THREADS, 2) verify_sm100_kernel(const VerifyFastParams p)
{
    extern __shared__ uint8_t fv_smem_raw[];
    const int b = blockIdx.x / p.h_v, h = blockIdx.x % p.h_v;
    if (!p.tree_ok[b]) return;
    const int base = p.node_offsets[b];
    const int T = p.node_offsets[b + 1] - base;
    if (T <= 0 || T > FV_T) return;   // larger trees never reach this kernel (host-side dispatch)

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(fv_smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    float *xs = reinterpret_cast<float *>(smem + SM_X);
    float *ys = reinterpret_cast<float *>(smem + SM_Y);
    float *a_s = reinterpret_cast<float *>(smem + SM_A);
    float *beta_s = reinterpret_cast<float *>(smem + SM_BETA);
    uint8_t *anc_s = smem + SM_ANC;
    uint8_t *depth_s = smem + SM_DEPTH;
    float *gram = reinterpret_cast<float *>(smem + SM_GRAM);
    float *ut = reinterpret_cast<float *>(smem + SM_UT);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM_TMEM);
    volatile uint32_t *flag = reinterpret_cast<volatile uint32_t *>(smem + SM_FLAG);
    const uint32_t mbar = sbase + SM_MBAR;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hk = h / (p.h_v / p.h_qk);

    if (warp == 0) tmem_alloc(sbase + SM_TMEM, FV_TMEM_COLS);
    if (tid == 32) {
        mbar_init(mbar, 1);
        *flag = 0;
    }

    // (1) k and q rows of the tree -> B operand tile (rows beyond T are zero-filled)
#pragma unroll
    for (int it = 0; it < (128 * 16) / FV_THREADS; ++it) {
        const int idx = it * FV_THREADS + tid;
        const int r = idx >> 4, c16 = idx & 15;
        const int node = r & 63;
        const bool valid = node < T;
        const __nv_bfloat16 *src = (r < 64 ? p.k : p.q) + ((size_t)(base + (valid ? node : 0)) * p.h_qk + hk) * FV_D + c16 * 8;
        cp_async_16(sbase + SM_B_KQ + sw128_offset(r, c16), src, valid);
    }
    // per-node metadata
    if (tid < T) {
        const int n = base + tid;
        const int d = p.depth[n];
        depth_s[tid] = (uint8_t)d;
        const uint16_t *row = p.anc + (size_t)n * p.max_depth;
        for (int a = 0; a < d; ++a) anc_s[tid * FV_MD + a] = (uint8_t)row[a];
        beta_s[tid] = __bfloat162float(p.beta[(size_t)n * p.h_v + h]);
    }

    // (2) state tile: fp32 -> bf16 hi + lo, written as the A operand.  A warp instruction covers
    // four rows; the eight lanes of a row each own one 16-byte piece of either K half.
    {
        const float *S = p.S0 + (size_t)(b * p.h_v + h) * FV_D * FV_D;
        const int r4 = lane >> 3, l8 = lane & 7;
        float4 x[4][4];   // [row i][kh*2 + half]
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = warp * 16 + i * 4 + r4;
            const float4 *src = reinterpret_cast<const float4 *>(S + (size_t)row * FV_D);
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                x[i][kh * 2 + 0] = __ldg(src + kh * 16 + l8 * 2 + 0);
                x[i][kh * 2 + 1] = __ldg(src + kh * 16 + l8 * 2 + 1);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = warp * 16 + i * 4 + r4;
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                const float4 u = x[i][kh * 2 + 0], w = x[i][kh * 2 + 1];
                const float f[8] = {u.x, u.y, u.z, u.w, w.x, w.y, w.z, w.w};
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float h0 = __bfloat162float(__float2bfloat16_rn(f[2 * e]));
                    const float h1 = __bfloat162float(__float2bfloat16_rn(f[2 * e + 1]));
                    hi[e] = pack_bf16(h0, h1);
                    lo[e] = pack_bf16(f[2 * e] - h0, f[2 * e + 1] - h1);
                }
                const uint32_t off = sw128_offset(row, kh * 8 + l8);
                *reinterpret_cast<uint4 *>(smem + SM_A_HI + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4 *>(smem + SM_A_LO + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
    }
    cp_async_wait_all();
    fence_proxy_async();   // generic-proxy writes of the operands become visible to the tensor core
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // (3) one thread issues the MMAs: P = S0.[K;Q]^T (hi then lo), Gram = [K;Q].K^T
    if (tid == 0) {
        const uint64_t a_hi = smem_desc_sw128(sbase + SM_A_HI), a_lo = smem_desc_sw128(sbase + SM_A_LO);
        const uint64_t b_kq = smem_desc_sw128(sbase + SM_B_KQ);
        constexpr uint32_t id_p = idesc_bf16(128, 128), id_g = idesc_bf16(128, 64);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem, a_hi + adv, b_kq + adv, id_p, ks > 0);
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem, a_lo + adv, b_kq + adv, id_p, 1);
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem + 128, b_kq + adv, b_kq + adv, id_g, ks > 0);
        }
        umma_commit(mbar);
    }

    // (4) while the tensor core works: decay from every path position to the node (suffix sums of g)
    if (tid < T) {
        const int d = depth_s[tid];
        float sfx = 0.f;
        for (int a = d - 1; a >= 0; --a) {
            xs[tid * FV_MD + a] = expf(sfx);
            sfx += __bfloat162float(p.g[(size_t)(base + anc_s[tid * FV_MD + a]) * p.h_v + h]);
        }
        a_s[tid] = expf(sfx);
    }

    // (5) wait for the MMAs (bounded: on expiry flag the error and fall through to the clean-up)
    {
        const long long t0 = clock64();
        bool done = mbar_try_wait(mbar, 0);
        while (!done) {
            if (clock64() - t0 > 400000000LL) break;   // ~0.2 s: far beyond any legitimate MMA latency
            done = mbar_try_wait(mbar, 0);
        }
        if (!done) *flag = 1;
    }
    tc_fence_after();
    __syncthreads();
    const bool timed_out = *flag != 0;

    if (!timed_out) {
        // (6) Gram block out of tensor memory: warp w reads lanes 32(w%4).., columns 128 + 32(w/4)..
        {
            const int row = (warp & 3) * 32 + lane;
            const int col0 = (warp >> 2) * 32;
            const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 128 + col0;
            uint32_t r0[16], r1[16];
            GDN_TMEM_LD16(taddr, r0);
            GDN_TMEM_LD16(taddr + 16, r1);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                gram[row * FV_GRAM_PITCH + col0 + j] = __uint_as_float(r0[j]);
                gram[row * FV_GRAM_PITCH + col0 + 16 + j] = __uint_as_float(r1[j]);
            }
        }
        __syncthreads();
        // (7) X and Y of Eq. 9 for real ancestors only
        for (int idx = tid; idx < T * FV_MD; idx += FV_THREADS) {
            const int i = idx / FV_MD, a = idx % FV_MD;
            const int d = depth_s[i];
            if (a < d) {
                const int j = anc_s[i * FV_MD + a];
                const float dec = xs[idx];
                ys[idx] = dec * gram[(64 + i) * FV_GRAM_PITCH + j];
                xs[idx] = beta_s[i] * dec * gram[i * FV_GRAM_PITCH + j];   // a = d-1 (self) is never read
            }
        }
        __syncthreads();

        // (8) substitution + output: thread c owns value component c of every node
        if (warp < 4) {
            const int c = tid;
            const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
            TOut *o = static_cast<TOut *>(p.o);
#pragma unroll 1
            for (int ch = 0; ch * 16 < T; ++ch) {
                uint32_t pk[16], pq[16];
                GDN_TMEM_LD16(trow + ch * 16, pk);
                GDN_TMEM_LD16(trow + 64 + ch * 16, pq);
                float vv[16];
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    const int i = ch * 16 + t;
                    vv[t] = i < T ? __bfloat162float(p.v[((size_t)(base + i) * p.h_v + h) * FV_D + c]) : 0.f;
                }
                tmem_wait_ld();
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    const int i = ch * 16 + t;
                    if (i < T) {
                        const int d = depth_s[i];
                        const uint8_t *an = anc_s + i * FV_MD;
                        const float *xi = xs + i * FV_MD, *yi = ys + i * FV_MD;
                        float sx = 0.f, sy = 0.f;
                        for (int a = 0; a < d - 1; ++a) {
                            const float uj = ut[an[a] * FV_D + c];
                            sx = fmaf(xi[a], uj, sx);
                            sy = fmaf(yi[a], uj, sy);
                        }
                        const float ai = a_s[i];
                        const float ui = beta_s[i] * (vv[t] - ai * __uint_as_float(pk[t])) - sx;
                        ut[i * FV_D + c] = ui;
                        const float out = p.scale * (fmaf(ai, __uint_as_float(pq[t]), sy) + yi[d - 1] * ui);
                        store_from_float(o + ((size_t)(base + i) * p.h_v + h) * FV_D + c, out);
                    }
                }
            }
        }
    } else if (tid == 0) {
        report_status(p.status_dev, GDN_ERR_TIMEOUT);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, FV_TMEM_COLS);
}

template <typename TOut>
cudaError_t launch_fast_typed(const gdn_shape_t &s, const VerifyFastParams &p, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(verify_sm100_kernel<TOut>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SM_ALLOC);
    if (e != cudaSuccess) return e;
    verify_sm100_kernel<TOut><<<s.n_seq * s.h_v, FV_THREADS, SM_ALLOC, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

bool verify_sm100_supported(const gdn_shape_t &s)
{
    return s.d_k == FV_D && s.d_v == FV_D && s.in_dtype == GDN_BF16 && s.max_tree_nodes <= FV_T &&
           s.max_depth <= FV_MD;
}

cudaError_t launch_verify_sm100(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                const void *v, const void *g, const void *beta,
                                const int32_t *node_offsets, void *o, const PlanPtrs &plan,
                                int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p{s.h_qk, s.h_v, s.max_depth, s.scale, S0,
                       static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k),
                       static_cast<const __nv_bfloat16 *>(v), static_cast<const __nv_bfloat16 *>(g),
                       static_cast<const __nv_bfloat16 *>(beta), node_offsets, o, plan.tree_ok, plan.depth,
                       plan.anc, status_dev};
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16>(s, p, stream);
    return launch_fast_typed<float>(s, p, stream);
}

}  // namespace gdn
