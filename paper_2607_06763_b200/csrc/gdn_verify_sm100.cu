// Tree-verify fast path for sm_100a: d_k = d_v = 128, bf16 inputs, trees of at most 64 nodes,
// root paths of at most 16 nodes.  Same mathematics as the generic kernel (the triangular form of
// Section 3.4.1 restricted to real ancestors, W S0 folded into the right-hand side as in
// Section 3.4.2), but the dense part runs on the 5th-generation tensor cores:
//
//   P  [d_v x 2T] = S0 [d_v x d_k] . [k_0;q_0;k_1;q_1;...]^T   (the S0 projections of Eq. 11 / Eq. 13: 86% of the FLOPs)
//   Gr [2T x 2T]  = [k;q rows] . [k;q rows]^T                  (k_i.k_j and q_i.k_j of Eq. 9; the .q columns are unused)
//
// Both are tcgen05.mma (kind::f16, bf16 operands, fp32 accumulators in tensor memory).  q and k
// are bf16 already; the fp32 state is split on the fly into two bf16 terms S0 = hi + lo
// (|S0 - hi - lo| <= 2^-16 |S0|), so P costs two accumulating MMA passes and keeps fp32-level
// accuracy.  Operand orientation: d_v on the TMEM lanes, nodes on the TMEM columns -- a thread then
// owns value component c and needs nothing from other components.
//
// Nodes are visited in depth-first (pre-order) order, prepared by the plan kernel.  In that order
// the proper ancestors of the current node are exactly the current stack, so the solve results
// u~ of the root path live in sixteen registers indexed by depth: the ancestor-masked forward
// substitution (Eq. 10 / 13) and the output (Eq. 11) of a node are straight-line FMAs against
// those registers, with the X / Y coefficients broadcast from shared memory, and u~ is never
// stored.  Warps 0-3 take the first half of the traversal, warps 4-7 the second half (after
// replaying the root path of their first node to rebuild its stack).
//
// One CTA per (tree, value head), 256 threads, about 106 KB of shared memory and 256 TMEM columns,
// so two CTAs share an SM: while one streams its 64 KB state tile from HBM the other computes.
#include "gdn_internal.cuh"

namespace gdn {

namespace {

constexpr int FV_THREADS = 256;
constexpr int FV_D = 128;           // d_k = d_v
constexpr int FV_T = 64;            // max nodes per tree
constexpr int FV_MD = 16;           // max nodes on a root path
constexpr int FV_TMEM_COLS = 256;   // P: columns [0,128) (2r: k_r, 2r+1: q_r), Gram: [128,256)
constexpr int FV_GRAM_PITCH = 65;   // floats per Gram row in shared memory (odd: conflict-free column writes)

// shared memory map (bytes from a 1024-byte aligned base); "r" is a depth-first position
constexpr int SM_A_HI = 0;                       // [2][128 rows][128 B], 128B-swizzled, K-major
constexpr int SM_A_LO = 32768;
constexpr int SM_B_KQ = 65536;                   // row 2r = k of node r, row 2r+1 = q of node r
constexpr int SM_GRAM = 0;                       // after the MMAs: fp32 [128][65] (columns = k_j) over A_HI/A_LO ...
constexpr int SM_V = 34816;                      // ... and the tree's v rows, bf16 [64][128]
constexpr int SM_X = 98304;                      // fp32 [64][16]: decay, then X coefficients
constexpr int SM_Y = SM_X + 4096;                // fp32 [64][16]: gathered g, then Y coefficients
constexpr int SM_ANCP = SM_Y + 4096;             // u8   [64][16]: positions of the root path
constexpr int SM_AB = SM_ANCP + 1024;            // float2 [64]: (total decay a_r, beta_r)
constexpr int SM_ORDER = SM_AB + 512;            // u8 [64] node id at position r
constexpr int SM_DPOS = SM_ORDER + FV_T;         // u8 [64] depth at position r (0 beyond T)
constexpr int SM_MBAR = SM_DPOS + FV_T;          // u64
constexpr int SM_TMEM = SM_MBAR + 8;             // u32
constexpr int SM_FLAG = SM_TMEM + 4;             // u32 (timeout flag)
constexpr int SM_BYTES = SM_FLAG + 4;
constexpr int SM_ALLOC = SM_BYTES + 1024;        // slack for the 1024-byte alignment of the base

struct VerifyFastParams {
    int h_qk, h_v;
    float scale;
    const float *S0;
    const __nv_bfloat16 *q, *k, *v, *g, *beta;
    const int32_t *node_offsets;
    void *o;
    const int32_t *tree_ok;
    const uint8_t *order8, *dpos8, *ancpos8;
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

#define GDN_TMEM_LD2(taddr, r0, r1) \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(taddr) : "memory")

// ---------------------------------------------------------------------------------------- kernel
// One node at depth D (D nodes on its root path).  st[a] holds u~ of the path node at depth a+1.
//   u~ = rhs - sum_{a<D-1} X[a] st[a]                       (forward substitution, Eq. 10 / 13)
//   ysum = sum_{a<D-1} Y[a] st[a] + Y[D-1] u~               (the Y term of Eq. 11)
template <int D>
__device__ __forceinline__ void node_step(float (&st)[FV_MD], const float *xr, const float *yr, float rhs,
                                          float &ysum)
{
    float acc0 = 0.f, acc1 = 0.f, y0 = 0.f, y1 = 0.f, ylast = 0.f;
#pragma unroll
    for (int q4 = 0; q4 * 4 < D; ++q4) {
        const float4 yv4 = *reinterpret_cast<const float4 *>(yr + q4 * 4);
        float4 xv4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q4 * 4 < D - 1) xv4 = *reinterpret_cast<const float4 *>(xr + q4 * 4);
        const float xv[4] = {xv4.x, xv4.y, xv4.z, xv4.w}, yv[4] = {yv4.x, yv4.y, yv4.z, yv4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int a = q4 * 4 + e;
            if (a < D - 1) {
                if (a & 1) { acc1 = fmaf(xv[e], st[a], acc1); y1 = fmaf(yv[e], st[a], y1); }
                else       { acc0 = fmaf(xv[e], st[a], acc0); y0 = fmaf(yv[e], st[a], y0); }
            } else if (a == D - 1) {
                ylast = yv[e];
            }
        }
    }
    const float u = rhs - (acc0 + acc1);
    st[D - 1] = u;
    ysum = fmaf(ylast, u, y0 + y1);
}

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
    float2 *ab_s = reinterpret_cast<float2 *>(smem + SM_AB);
    uint8_t *ancp = smem + SM_ANCP;
    uint8_t *order_s = smem + SM_ORDER;
    uint8_t *dpos_s = smem + SM_DPOS;
    float *gram = reinterpret_cast<float *>(smem + SM_GRAM);
    const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(smem + SM_V);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM_TMEM);
    volatile uint32_t *flag = reinterpret_cast<volatile uint32_t *>(smem + SM_FLAG);
    const uint32_t mbar = sbase + SM_MBAR;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hk = h / (p.h_v / p.h_qk);

    // (1) state tile loads first (the longest latency of the prologue): a warp instruction covers
    // four rows; the eight lanes of a row each own one 16-byte bf16 piece of either K half.
    const int r4 = lane >> 3, l8 = lane & 7;
    float4 x[4][4];   // [row i][kh*2 + half]
    {
        const float *S = p.S0 + (size_t)(b * p.h_v + h) * FV_D * FV_D;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 *src = reinterpret_cast<const float4 *>(S + (size_t)(warp * 16 + i * 4 + r4) * FV_D);
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                x[i][kh * 2 + 0] = __ldg(src + kh * 16 + l8 * 2 + 0);
                x[i][kh * 2 + 1] = __ldg(src + kh * 16 + l8 * 2 + 1);
            }
        }
    }

    if (warp == 0) tmem_alloc(sbase + SM_TMEM, FV_TMEM_COLS);
    if (tid == 32) {
        mbar_init(mbar, 1);
        *flag = 0;
    }
    // (2) depth-first tables of this tree
    if (tid < FV_T) {
        int d = 0, node = 0;
        uint4 row = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
        if (tid < T) {
            node = p.order8[base + tid];
            d = p.dpos8[base + tid];
            row = __ldg(reinterpret_cast<const uint4 *>(p.ancpos8 + (size_t)(base + tid) * 16));
        }
        order_s[tid] = (uint8_t)node;
        dpos_s[tid] = (uint8_t)d;
        *reinterpret_cast<uint4 *>(ancp + tid * 16) = row;
    }
    __syncthreads();

    // (3) k and q rows in depth-first order -> B operand tile (rows beyond T are zero-filled)
#pragma unroll
    for (int it = 0; it < (128 * 16) / FV_THREADS; ++it) {
        const int idx = it * FV_THREADS + tid;
        const int r = idx >> 4, c16 = idx & 15;
        const int pos = r >> 1;
        const bool valid = pos < T;
        const int node = valid ? order_s[pos] : 0;
        const __nv_bfloat16 *src = ((r & 1) ? p.q : p.k) + ((size_t)(base + node) * p.h_qk + hk) * FV_D + c16 * 8;
        cp_async_16(sbase + SM_B_KQ + sw128_offset(r, c16), src, valid);
    }

    // (4) fp32 -> bf16 hi + lo, written as the A operand
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
    cp_async_wait_all();
    fence_proxy_async();   // generic-proxy writes of the operands become visible to the tensor core
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // (5) one thread issues the MMAs: P = S0.[k;q]^T (hi then lo), Gram = [k;q].[k;q]^T
    if (tid == 0) {
        const uint64_t a_hi = smem_desc_sw128(sbase + SM_A_HI), a_lo = smem_desc_sw128(sbase + SM_A_LO);
        const uint64_t b_kq = smem_desc_sw128(sbase + SM_B_KQ);
        constexpr uint32_t id = idesc_bf16(128, 128);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem, a_hi + adv, b_kq + adv, id, ks > 0);
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem, a_lo + adv, b_kq + adv, id, 1);
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
            umma_bf16(tmem + 128, b_kq + adv, b_kq + adv, id, ks > 0);
        }
        umma_commit(mbar);
    }

    // (6) while the tensor core works: g of every path node, then the decay from each path
    // position to the node as exp of a suffix sum (= a_i / a_j of Eq. 9 without cancellation)
    for (int idx = tid; idx < FV_T * FV_MD; idx += FV_THREADS) {
        const int r = idx >> 4, a = idx & 15;
        float gv = 0.f;
        if (a < dpos_s[r]) gv = __bfloat162float(p.g[(size_t)(base + order_s[ancp[idx]]) * p.h_v + h]);
        ys[idx] = gv;
    }
    float beta_r = 0.f;
    if (tid < T) beta_r = __bfloat162float(p.beta[(size_t)(base + order_s[tid]) * p.h_v + h]);
    __syncthreads();
    for (int idx = tid; idx < FV_T * FV_MD; idx += FV_THREADS) {
        const int r = idx >> 4, a = idx & 15;
        const int d = dpos_s[r];
        if (a < d) {
            float sfx = 0.f;
            for (int u = a + 1; u < d; ++u) sfx += ys[r * FV_MD + u];
            xs[idx] = expf(sfx);
        }
    }
    if (tid < T) {
        float tot = 0.f;
        for (int u = 0; u < dpos_s[tid]; ++u) tot += ys[tid * FV_MD + u];
        ab_s[tid] = make_float2(expf(tot), beta_r);
    }

    // (7) wait for the MMAs (bounded: on expiry flag the error and fall through to the clean-up)
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
        // (8) the operand tiles are free now: fetch the tree's v rows over them (depth-first order),
        // and move the k-columns of the Gram block out of tensor memory
#pragma unroll
        for (int it = 0; it < (FV_T * 16) / FV_THREADS; ++it) {
            const int idx = it * FV_THREADS + tid;
            const int r = idx >> 4, c16 = idx & 15;
            const bool valid = r < T;
            const int node = valid ? order_s[r] : 0;
            cp_async_16(sbase + SM_V + r * 256 + c16 * 16, p.v + ((size_t)(base + node) * p.h_v + h) * FV_D + c16 * 8,
                        valid);
        }
        {
            const int row = (warp & 3) * 32 + lane;
            const int half = warp >> 2;   // TMEM columns 128 + 64*half .. : k_j for j = 32*half ..
            const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 128 + half * 64;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                uint32_t r0[16], r1[16];
                GDN_TMEM_LD16(taddr + part * 32, r0);
                GDN_TMEM_LD16(taddr + part * 32 + 16, r1);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    gram[row * FV_GRAM_PITCH + half * 32 + part * 16 + j] = __uint_as_float(r0[2 * j]);
                    gram[row * FV_GRAM_PITCH + half * 32 + part * 16 + 8 + j] = __uint_as_float(r1[2 * j]);
                }
            }
        }
        __syncthreads();
        // (9) X and Y of Eq. 9 for real ancestors only
        for (int idx = tid; idx < FV_T * FV_MD; idx += FV_THREADS) {
            const int r = idx >> 4, a = idx & 15;
            if (a < dpos_s[r]) {
                const int j = ancp[idx];
                const float dec = xs[idx];
                ys[idx] = dec * gram[(2 * r + 1) * FV_GRAM_PITCH + j];
                xs[idx] = ab_s[r].y * dec * gram[(2 * r) * FV_GRAM_PITCH + j];   // a = d-1 (self) is never read
            }
        }
        cp_async_wait_all();
        __syncthreads();

        // (10) depth-first sweep: thread c owns value component c; warps 0-3 take positions
        // [0, r_mid), warps 4-7 rebuild the stack of r_mid's root path and take [r_mid, T)
        {
            const int c = tid & 127;
            const uint32_t trow = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            TOut *o = static_cast<TOut *>(p.o);
            float st[FV_MD];
#pragma unroll
            for (int a = 0; a < FV_MD; ++a) st[a] = 0.f;
            const int r_mid = (T + 1) >> 1;
            const bool second = warp >= 4;
            const int n_pre = (second && r_mid < T) ? dpos_s[r_mid] - 1 : 0;
            const int r_begin = second ? r_mid : 0, r_end = second ? T : r_mid;
#pragma unroll 1
            for (int it = -n_pre; it < r_end - r_begin; ++it) {
                const bool store = it >= 0;
                const int r = store ? r_begin + it : ancp[r_mid * FV_MD + (it + n_pre)];
                uint32_t pk, pq;
                GDN_TMEM_LD2(trow + 2 * r, pk, pq);
                const float2 ab = ab_s[r];
                const float v = __bfloat162float(vs[r * FV_D + c]);
                const int d = dpos_s[r];
                const float *xr = xs + r * FV_MD, *yr = ys + r * FV_MD;
                tmem_wait_ld();
                const float rhs = ab.y * (v - ab.x * __uint_as_float(pk));
                float ysum = 0.f;
                switch (d) {
                case 1: node_step<1>(st, xr, yr, rhs, ysum); break;
                case 2: node_step<2>(st, xr, yr, rhs, ysum); break;
                case 3: node_step<3>(st, xr, yr, rhs, ysum); break;
                case 4: node_step<4>(st, xr, yr, rhs, ysum); break;
                case 5: node_step<5>(st, xr, yr, rhs, ysum); break;
                case 6: node_step<6>(st, xr, yr, rhs, ysum); break;
                case 7: node_step<7>(st, xr, yr, rhs, ysum); break;
                case 8: node_step<8>(st, xr, yr, rhs, ysum); break;
                case 9: node_step<9>(st, xr, yr, rhs, ysum); break;
                case 10: node_step<10>(st, xr, yr, rhs, ysum); break;
                case 11: node_step<11>(st, xr, yr, rhs, ysum); break;
                case 12: node_step<12>(st, xr, yr, rhs, ysum); break;
                case 13: node_step<13>(st, xr, yr, rhs, ysum); break;
                case 14: node_step<14>(st, xr, yr, rhs, ysum); break;
                case 15: node_step<15>(st, xr, yr, rhs, ysum); break;
                case 16: node_step<16>(st, xr, yr, rhs, ysum); break;
                default: break;
                }
                if (store) {
                    const float out = p.scale * fmaf(ab.x, __uint_as_float(pq), ysum);
                    store_from_float(o + ((size_t)(base + order_s[r]) * p.h_v + h) * FV_D + c, out);
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
    VerifyFastParams p{s.h_qk, s.h_v, s.scale, S0,
                       static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k),
                       static_cast<const __nv_bfloat16 *>(v), static_cast<const __nv_bfloat16 *>(g),
                       static_cast<const __nv_bfloat16 *>(beta), node_offsets, o, plan.tree_ok, plan.order8,
                       plan.dpos8, plan.ancpos8, status_dev};
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16>(s, p, stream);
    return launch_fast_typed<float>(s, p, stream);
}

}  // namespace gdn
