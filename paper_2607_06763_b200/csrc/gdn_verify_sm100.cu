// Tree-verify fast path for sm_100a: d_k = d_v = 128, bf16 inputs, root paths of at most 16 nodes, at most 64 nodes
// per unit of work (larger trees are cut into ancestor-closed groups, each a unit of its own).  It evaluates the
// triangular form of Section 3.4.1 (Eq. 9-11) restricted to real ancestors, with the W S0 term folded into the
// right-hand side as in Section 3.4.2, and turns all of the per-component work into dense contractions on the
// 5th-generation tensor cores (tcgen05.mma, bf16 operands, fp32 accumulators in tensor memory):
//
//   (1) P  [d_v x 2T] = S0 [d_v x d_k] . [k rows; q rows]^T          the S0 projections of Eq. 11 / Eq. 13
//       Gr [2T x T]   = [k rows; q rows] . [k rows]^T                k_i.k_j and q_i.k_j of Eq. 9
//   (2) D  [d_v x T]  = R^T [d_v x T] . Z^T [T x T]                  the whole masked solve + output
//
// where r_j = beta_j (v_j - a_j S0^T k_j) is the folded right-hand side and row i of Z is
// z_i^T = y_i^T (I + X_path(i))^-1: because the ancestors of a node form a chain, the inverse restricted to one
// root path is a back-substitution with at most 16 unknowns that each node can run on its own (four threads per
// node, no dependence between nodes).  Then
//   o_i = scale (a_i S0^T q_i + sum_{j on the root path of i} Z_ij r_j),
// which is Eq. 11 with U - W S0 eliminated; no per-component sequential substitution is left.
// fp32 quantities that feed the tensor cores are split into two bf16 terms (x = hi + lo, |x - hi - lo| <= 2^-16 |x|):
// S0 for (1), R and Z for (2); the lo.lo term of (2) is dropped.
//
// Operand orientation: d_v on the TMEM lanes, nodes on the TMEM columns, so every thread of a warp owns one value
// component.  256 threads, about 112 KB of shared memory and 256 TMEM columns per CTA, so two CTAs share an SM.
// One persistent kernel: a software pipeline across the units of a CTA, TMA tiles on mbarriers for trees that fit
// one unit (optionally with the commit of the previous step fused in front), row gathers through the plan's node
// table for the groups of larger trees.
#include <cuda.h>   // CUtensorMap and the cuTensorMapEncodeTiled prototype (resolved at run time, no libcuda link)

#include "gdn_internal.cuh"
#include "gdn_replay.cuh"

namespace gdn {

namespace {

constexpr int FV_THREADS = 256;
constexpr int FV_D = 128;           // d_k = d_v
constexpr int FV_T = 64;            // max nodes per tree
constexpr int FV_MD = 16;           // max nodes on a root path
constexpr int FV_TMEM_COLS = 256;   // P: columns [0,128); D: [128,192); Gram block of the unit to come: [192,256)

// shared memory map (bytes from a 1024-byte aligned base)
constexpr int SM_A_HI = 0;                       // S0 hi: [2][128 rows][128 B], 128B-swizzled, K-major
constexpr int SM_A_LO = 32768;                   // S0 lo
constexpr int SM_B_KQ = 65536;                   // k and q rows, same layout: rows 0..63 = k, 64..127 = q
// after the first MMA group the operand tiles are dead and are reused:
constexpr int SM_GRAM = 0;                       // fp32 [128][64]: four-column piece c of row r at position c ^ (r & 15)
constexpr int SM_RT_HI = 0;                      // then R^T hi: [128 rows = components][64 nodes] bf16, swizzled
constexpr int SM_RT_LO = 16384;                  //      R^T lo
constexpr int SM_VE = 40960;                     // v rows of the tree, bf16 [64][128]: they land here at the top of a unit (free
                                                 // until the state operand is written) and move into registers before that
constexpr int SM_Z_HI = 49152;                   // Z hi: [64 rows = nodes i][64 nodes j] bf16, swizzled
constexpr int SM_Z_LO = 57344;                   // Z lo
constexpr int SM_X = 98304;                      // fp32 [64][16]  X(i, t-th path node)
constexpr int SM_Y = SM_X + 4096;                // fp32 [64][16]  Y(i, t-th path node), node itself included
constexpr int SM_ANC = SM_Y + 4096;              // u8   [64][16]  root-path node ids (0xFF = unused)
constexpr int SM_GAB = SM_ANC + 1024;            // float4 [64]: (G_i = log a_i, a_i, beta_i, g_i)
constexpr int SM_DEPTH = SM_GAB + 1024;          // u8 [64] (0 beyond T)
constexpr int SM_PATH = SM_DEPTH + FV_T;         // fused commit, two slots of 384 B: int [16] path node ids, int length (0 = no
                                                 // replay), int first node of the tree; at +128 float4 [16] (A_t = decay of the
                                                 // path up to and including step t, beta_t, alpha_t, 1 / A_t)
constexpr int SM_PATH_SLOT = 384;
constexpr int SM_PK = 32768;                     // fused commit: k rows of the accepted path, bf16 [16][128], parked in the
constexpr int SM_PV = 36864;                     // state-operand area until the replay is over; v rows likewise
constexpr int SM_TABLE2 = SM_PATH + 2 * SM_PATH_SLOT;   // second copy of ANC / GAB / DEPTH (2112 B)
constexpr int SM_TABLE_STRIDE = SM_TABLE2 - SM_ANC;   // table buffer tb lives SM_TABLE_STRIDE * tb further on
constexpr int SM_MBAR = SM_TABLE2 + 2176;        // 5 x u64: Gram done, P done, D done, k/q tile landed, v tile landed
constexpr int SM_TMEM = SM_MBAR + 40;            // u32
constexpr int SM_FLAG = SM_TMEM + 4;             // u32 (timeout flag)
constexpr int SM_PAR = SM_FLAG + 4;              // s8 [64] parent[] of the tree whose tables are being built
constexpr int SM_BAD = SM_PAR + FV_T;            // int [2], tree of table buffer tb was rejected
constexpr int SM_VN2 = SM_BAD + 8;               // grouped mode: u16 [2][64] node id of virtual index u (per table buffer)
constexpr int SM_BYTES = SM_VN2 + 2 * 2 * FV_T;
constexpr int SM_ALLOC = SM_BYTES + 1024;        // slack for the 1024-byte alignment of the base

struct VerifyFastParams {
    // TMA descriptors of the packed k, q, v tensors viewed as [N][heads][128] bf16 (not used by the grouped mode)
    alignas(64) CUtensorMap tm_k;
    alignas(64) CUtensorMap tm_q;
    alignas(64) CUtensorMap tm_v;
    int h_qk, h_v;
    int n_units;        // n_seq * h_v (grouped mode: an upper bound that only sizes the grid)
    int prefetch_dist;  // a CTA warms L2 for unit blockIdx.x + prefetch_dist (about one wave ahead)
    float scale;
    const float *S0;
    const __nv_bfloat16 *q, *k, *v, *g, *beta;
    const int32_t *node_offsets;
    const int32_t *parent;                             // trees of at most 64 nodes: the kernel builds the metadata itself
    int n_seq, total_nodes, max_tree_nodes, max_depth;
    void *o;
    const uint8_t *depth;
    const uint8_t *anc8;
    int32_t *status_dev;
    // grouped verification of trees with more than 64 nodes (only read by the GROUPED instantiation)
    int groups_per_tree, anc_stride;                   // upper bound of the groups of a tree (sizes the grid); entries
                                                       // per row of anc16
    const uint16_t *anc16, *dfs_node;
    const uint4 *unit_list;                            // one record per group (see the workspace layout)
    const int32_t *unit_count;                         // [0] records in the list, [1] plan_magic of the plan's shape
    int unit_capacity, plan_magic;                     // what the list can hold; what [1] has to read
    const uint8_t *dfs_depth, *dfs_anc8;
    // fused commit of the previous step's accepted paths (only read by the FUSED instantiation)
    float *S_rw;                                       // same tensor as S0, written in place
    const __nv_bfloat16 *pk, *pv, *pg, *pbeta;         // the previous tree's k, v, g, beta
    const int32_t *pparent, *pnode_offsets, *path, *path_offsets;
    // Padded layout of Section 3.4.2 (persistent kernel; t_pad = 0: ragged packing by node_offsets[]): slot b keeps
    // its nodes in rows b * t_pad .. and carries tree b % n_trees, whose parent[] row and node count are shared by
    // all the slots (layers) of that tree; the accepted paths are per tree as well.
    int t_pad, n_trees, pt_pad, path_stride;
    const int32_t *n_nodes, *pn_nodes, *path_len;
    int raw_gates;                                     // g / beta arrive as raw gate inputs ("scalars" stage on chip)
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
// Ask L2 to fetch `bytes` (a multiple of 16) starting at `p`; nothing waits for it.
__device__ __forceinline__ void prefetch_l2_bulk(const void *p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
// TMA: one thread announces the bytes a barrier has to see, then issues tiled loads that complete on it.
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar)
                 : "memory");
}
// The mbarrier receives one arrival from this thread once all cp.async it has issued so far have landed (the
// barrier's expected count has to include that arrival).
__device__ __forceinline__ void cp_async_arrive_on(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
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
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
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

#define GDN_TMEM_LD32(taddr, r)                                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                  \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                  \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                 \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),      \
                   "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),  \
                   "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),            \
                   "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),            \
                   "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])             \
                 : "r"(taddr)                                                                                \
                 : "memory")

// Byte offset of 16-byte piece `c16` (0..7) of row `r` in a one-atom-wide ([rows][128 B]) swizzled tile.
__device__ __forceinline__ uint32_t sw128_row_offset(int r, int c16)
{
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c16 ^ (r & 7)) << 4));
}

// One lane of a converged warp (the branch around it stays warp-uniform, so that descriptors can live in
// uniform registers).
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}

// Bounded wait on an mbarrier phase; returns false if it expired.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    const long long t0 = clock64();
    bool done = mbar_try_wait(bar, parity);
    while (!done) {
        if (clock64() - t0 > 400000000LL) break;   // ~0.2 s: far beyond any legitimate MMA latency
        done = mbar_try_wait(bar, parity);
    }
    return done;
}

// Two fp32 values -> packed bf16 pair of the leading parts and packed bf16 pair of the remainders.
__device__ __forceinline__ void split_pack_bf16(float x0, float x1, uint32_t &hi, uint32_t &lo)
{
    hi = pack_bf16(x0, x1);
    const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xFFFF0000u);
    lo = pack_bf16(x0 - h0, x1 - h1);
}
__device__ __forceinline__ void split_bf16(float x, float &hi, float &lo)
{
    hi = __bfloat162float(__float2bfloat16_rn(x));
    lo = x - hi;
}

// ---------------------------------------------------------------------------------------- kernel
// The k/q tile holds the k rows first and the q rows second (rows i and 64 + i), so P has p^k in columns 0..63 and
// p^q in columns 64..127, and the Gram block needs only N = 64.
// FUSED: Eq. 7 is replayed along the previous step's accepted path on the state tile while it sits in registers
// -- per row c, s_c <- alpha s_c + k beta (v_c - alpha k.s_c), the eight lanes that share a row reducing k.s_c with
// three shuffles -- the tile is written back as the only state write of the step, and the new tree is verified
// against it.
// A CTA keeps its tensor memory and walks over the units blockIdx.x, blockIdx.x + gridDim.x, ...  Nothing a unit
// can know in advance is waited for inside it: the next unit's k/q tile streams into the operand tile as soon as the
// first MMA group has released it, its Gram block is issued at the end of the current unit into spare TMEM columns,
// and its per-node tables, decay tables and accepted path are fetched in stages, each global load one phase before
// its value is used.  The state tile is asked for at the top of the unit and is needed only after the Gram /
// coefficient phases; the v rows land by TMA in an area that is free until the state operand is written.
// SMALL (every tree of the call has at most 32 nodes): the R and output phases skip the 16-node pieces beyond the tree.
// GROUPED (trees of more than 64 nodes, cut into ancestor-closed groups by the plan kernel): a unit is (tree, value
// head, group); it is verified as a virtual tree of the <= 15 proper ancestors of the group's first node followed by
// the group's own nodes.  The rows of a virtual tree are not contiguous, so its k/q/v rows are gathered with
// cp.async (completing on the same mbarriers as the TMA tiles otherwise), its tables come from the plan, and
// outputs are stored for the group's own nodes only.  The units are the records of the plan's unit list (one per
// real group, the groups of a tree next to one another) times the heads: the five or so groups of a (tree, head) run
// on neighbouring CTAs at about the same time, so the state tile crosses HBM once, and the work spreads evenly over
// the CTAs whatever the tree sizes.
template <typename TOut, bool FUSED, bool SMALL, bool PADDED, bool GROUPED>
__global__ void __launch_bounds__(FV_THREADS, 2) verify_sm100_persistent_kernel(const __grid_constant__ VerifyFastParams p)
{
    static_assert(!GROUPED || (!FUSED && !SMALL), "the grouped mode is verification only");
    extern __shared__ uint8_t fv_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(fv_smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    float *xs = reinterpret_cast<float *>(smem + SM_X);
    float *ys = reinterpret_cast<float *>(smem + SM_Y);
    float *gram = reinterpret_cast<float *>(smem + SM_GRAM);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM_TMEM);
    volatile uint32_t *flag = reinterpret_cast<volatile uint32_t *>(smem + SM_FLAG);
    const uint32_t mbar_g = sbase + SM_MBAR, mbar_p = mbar_g + 8, mbar_d = mbar_g + 16;
    const uint32_t mbar_kq = mbar_g + 24, mbar_v = mbar_g + 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r4 = lane >> 3, l8 = lane & 7;
    // The asynchronous work of a unit is issued by one elected lane each of four warps, so that no single warp
    // carries all of it: warp 0 the projection MMA group, warp 1 the D group, warp 2 the Gram block of the unit to
    // come, warp 3 the TMA loads.  Every issuer commits its own MMAs to an mbarrier.
    constexpr int W_MMA_P = 0, W_MMA_D = 1, W_MMA_G = 2, W_TMA = 3;
    auto tbl_thread_g = [&]() -> bool { return tid >= FV_T && tid < 2 * FV_T; };   // thread FV_T + i keeps node i's tables

    if (warp == 0) tmem_alloc(sbase + SM_TMEM, FV_TMEM_COLS);
    if (tid == 32) {
        mbar_init(mbar_g, 1);
        mbar_init(mbar_p, 1);
        mbar_init(mbar_d, 1);
        mbar_init(mbar_kq, GROUPED ? FV_THREADS : 1);   // gathered rows: every thread arrives once its copies have landed
        mbar_init(mbar_v, GROUPED ? FV_THREADS : 1);
        *flag = 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // warp-uniform by construction
    // Launched with programmatic stream serialization: everything above overlaps the tail of the kernel in front
    // (the previous call, or the plan kernel); nothing that is computed from memory may run before that kernel's
    // writes are visible.  L2 can be asked for the first unit's state tile meanwhile (a prefetch consumes nothing).
    if (!GROUPED && tid < 4 && (int)blockIdx.x < p.n_units)
        prefetch_l2_bulk(p.S0 + (size_t)blockIdx.x * FV_D * FV_D + (size_t)tid * 4096, 16384);
    // ... and for the rows of the first unit's tree.  Their place may depend on node_offsets[], which the kernel in
    // front may still be writing: the value read here only steers prefetches (clamped to the tensors), it is read
    // again behind the dependency wait before anything is computed from it.
    if (!GROUPED && (int)blockIdx.x < p.n_units && tid >= 128 && tid < 128 + FV_T) {
        const int ub = (int)blockIdx.x / p.h_v, uh = (int)blockIdx.x % p.h_v, uhk = uh / (p.h_v / p.h_qk);
        const int row = ((PADDED && p.t_pad) ? ub * p.t_pad : __ldg(p.node_offsets + ub)) + tid - 128;
        if (row >= 0 && row < p.total_nodes) {
            prefetch_l2_bulk(p.v + ((size_t)row * p.h_v + uh) * FV_D, 256);
            prefetch_l2_bulk(p.k + ((size_t)row * p.h_qk + uhk) * FV_D, 256);
            prefetch_l2_bulk(p.q + ((size_t)row * p.h_qk + uhk) * FV_D, 256);
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.g + (size_t)row * p.h_v + uh));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.beta + (size_t)row * p.h_v + uh));
        }
    }
    signed char *par_s = reinterpret_cast<signed char *>(smem + SM_PAR);
    volatile int *bad_s = reinterpret_cast<volatile int *>(smem + SM_BAD);

    // unit -> (tree, head, first node, size); a unit whose node_offsets[] are inconsistent (reported) or whose tree
    // is empty is skipped.  parent[] itself is checked when the unit's tables are built.
    // A CTA walks the units blockIdx.x, blockIdx.x + gridDim.x, ...: the indices of a unit follow from those of the
    // unit before by additions and carries, so that the integer divisions by the head and group counts (a few dozen
    // instructions each, for every thread) are paid once per CTA and not once per unit.
    // Trees of at most 64 nodes: unit = slot b * h_v + head h.  GROUPED: unit = (layer b * E + record grp) * h_v + h,
    // where E is the number of records in the plan's unit list (one per group; known behind the dependency wait) and
    // `layer` counts the repetitions of the n_trees shared trees in the padded layout (always 0 otherwise).
    struct Cursor { int u, b, h, grp; };
    int n_units = GROUPED ? 0 : p.n_units;
    int n_records = 1, gstep_h = 0, gstep_e = 0, gstep_l = 0;   // GROUPED, set behind the dependency wait
    const int ratio = p.h_v / p.h_qk;
    const int ratio_shift = (ratio & (ratio - 1)) == 0 ? 31 - __clz(ratio) : -1;
    auto hk_of = [&](int h_) -> int { return ratio_shift >= 0 ? h_ >> ratio_shift : h_ / ratio; };
    auto tree_of = [&](int b_) -> int { return p.n_trees == 1 ? 0 : b_ % p.n_trees; };   // padded layout only
    const int step_h = (int)gridDim.x % p.h_v, step_b = (int)gridDim.x / p.h_v;
    auto cursor_at = [&](int u) -> Cursor {
        Cursor c;
        c.u = u;
        c.h = u % p.h_v;
        const int t = u / p.h_v;
        c.grp = GROUPED ? t % n_records : 0;
        c.b = GROUPED ? t / n_records : t;
        return c;
    };
    auto advance = [&](Cursor &c) {
        c.u += (int)gridDim.x;
        if constexpr (GROUPED) {
            c.h += gstep_h;
            const int carry_h = c.h >= p.h_v ? 1 : 0;
            c.h -= carry_h ? p.h_v : 0;
            c.grp += gstep_e + carry_h;
            const int carry_e = c.grp >= n_records ? 1 : 0;
            c.grp -= carry_e ? n_records : 0;
            c.b += gstep_l + carry_e;
        } else {
            c.h += step_h;
            const int carry_h = c.h >= p.h_v ? 1 : 0;
            c.h -= carry_h ? p.h_v : 0;
            c.b += step_b + carry_h;
        }
    };
    // The loads a decode needs are issued by decode_load() and looked at by decode() / decode_g() later (the unit after
    // next is asked for at the top of a unit and decoded in its middle), so that no thread waits for them.
    struct DecodeRaw { int lo, hi; uint4 rec; };
    auto decode_load = [&](const Cursor &c) -> DecodeRaw {
        DecodeRaw r{0, 0, make_uint4(0u, 0u, 0u, 0u)};
        if (c.u >= n_units) return r;
        const int ub = c.b;
        if constexpr (GROUPED) {
            r.rec = p.unit_list[c.grp];   // written by the plan kernel in front of this grid: no read-only path
        } else if (PADDED && p.t_pad) {
            r.lo = p.n_nodes[tree_of(ub)];
        } else {
            r.lo = p.node_offsets[ub];
            r.hi = p.node_offsets[ub + 1];
        }
        return r;
    };
    auto decode = [&](const Cursor &c, const DecodeRaw &raw, int &ub, int &uh, int &uhk, int &ubase, int &uT, int &upar) -> bool {
        if (c.u >= n_units) return false;
        ub = c.b;
        uh = c.h;
        uhk = hk_of(uh);
        bool off_ok;
        if (PADDED && p.t_pad) {   // padded layout: rows of the slot, node count and parent[] row of its tree
            const int tree = tree_of(ub);
            ubase = ub * p.t_pad;
            uT = raw.lo;
            upar = tree * p.t_pad;
            off_ok = uT >= 0 && uT <= FV_T && uT <= p.t_pad;
        } else {
            ubase = raw.lo;
            const int uend = raw.hi;
            uT = uend - ubase;
            upar = ubase;
            off_ok = ubase >= 0 && uT >= 0 && uT <= FV_T && uT <= p.max_tree_nodes && uend <= p.total_nodes;
            if (ub == 0) off_ok = off_ok && ubase == 0;
            if (ub == p.n_seq - 1) off_ok = off_ok && uend == p.total_nodes;
        }
        if (!off_ok && tid == 0) report_status(p.status_dev, GDN_ERR_TREE);
        const bool tree_good = off_ok && uT > 0;
        if (FUSED && !tree_good) {
            // the commit of the previous step does not depend on the new tree: the unit runs as a tree of no
            // nodes (every node masked, nothing stored), so that its accepted path is still replayed
            ubase = 0;
            uT = 0;
            upar = 0;
            return true;
        }
        return tree_good;
    };
    // GROUPED: unit -> (tree, head, group).  pb = first row of the tree in the plan's tables, g0 = first depth-first
    // position of the group, n_prefix = proper ancestors of its first node (virtual indices 0 .. n_prefix - 1),
    // first = node at position g0; ident: a tree of at most 64 nodes inside a grouped call (identity numbering).
    struct GroupX { int pb, g0, n_prefix, first; bool ident; };
    auto decode_g = [&](const Cursor &c, const DecodeRaw &raw, int &ub, int &uh, int &uhk, int &ubase, int &uT, GroupX &gx) -> bool {
        if (c.u >= n_units) return false;
        const int tree = (int)raw.rec.x;
        uh = c.h;
        uhk = hk_of(uh);
        if (PADDED && p.t_pad) {   // slot = layer * n_trees + tree
            ub = c.b * p.n_trees + tree;
            ubase = ub * p.t_pad;
            gx.pb = tree * p.t_pad;
        } else {
            ub = tree;
            ubase = (int)raw.rec.y;   // checked by the plan kernel (a tree with bad offsets has no record)
            gx.pb = ubase;
        }
        const uint2 gi = make_uint2(raw.rec.z, raw.rec.w);
        const int own = (int)(gi.x >> 16);
        if (own == 0) return false;   // no such group (or the plan rejected the tree, which it has reported)
        gx.g0 = (int)(gi.x & 0xFFFFu);
        gx.ident = (gi.y & 0xFFFFu) == 0xFFFFu;
        gx.n_prefix = gx.ident ? 0 : (int)(gi.y & 0xFFFFu);
        gx.first = (int)(gi.y >> 16);
        uT = gx.n_prefix + own;
        return true;
    };
    // node id of virtual index u (< T) of a group, from the plan
    auto vnode_global = [&](const GroupX &gx, int u) -> int {
        if (gx.ident) return u;
        if (u < gx.n_prefix) return (int)__ldg(p.anc16 + (size_t)(gx.pb + gx.first) * p.anc_stride + u);
        return (int)__ldg(p.dfs_node + gx.pb + gx.g0 + u - gx.n_prefix);
    };
    // table entries of virtual index tnode: node id, depth, root path in virtual indices
    auto lookup_tables_g = [&](const GroupX &gx, int uT, int &node, int &d, uint4 &row) {
        node = 0;
        d = 0;
        row = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
        if (tbl_thread_g() && tid - FV_T < uT) {
            const int t = tid - FV_T;
            if (gx.ident) {
                node = t;
                d = p.depth[gx.pb + t];
                row = __ldg(reinterpret_cast<const uint4 *>(p.anc8 + (size_t)(gx.pb + t) * 16));
            } else if (t < gx.n_prefix) {   // an ancestor of the group's first node: its path is 0..t
                node = vnode_global(gx, t);
                d = t + 1;
                const uint32_t all[4] = {0x03020100u, 0x07060504u, 0x0B0A0908u, 0x0F0E0D0Cu};
                uint32_t w[4];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int keep = d - 4 * q4;   // bytes of this word that are on the path
                    w[q4] = keep >= 4 ? all[q4] : keep <= 0 ? 0xFFFFFFFFu : (all[q4] | (0xFFFFFFFFu << (8 * keep)));
                }
                row = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                const int r = gx.pb + gx.g0 + t - gx.n_prefix;
                node = (int)__ldg(p.dfs_node + r);
                d = p.dfs_depth[r];
                row = __ldg(reinterpret_cast<const uint4 *>(p.dfs_anc8 + (size_t)r * 16));
            }
        }
    };
    auto put_tables_g = [&](int uT, int tb, int node, int d, uint4 row, uint32_t g_bits, uint32_t be_bits) {
        if (tbl_thread_g()) {
            const int t = tid - FV_T;
            const bool on = t < uT;
            (smem + SM_DEPTH + tb * SM_TABLE_STRIDE)[t] = (uint8_t)(on ? d : 0);
            *reinterpret_cast<uint4 *>(smem + SM_ANC + tb * SM_TABLE_STRIDE + t * 16) = row;
            reinterpret_cast<float4 *>(smem + SM_GAB + tb * SM_TABLE_STRIDE)[t] =
                make_float4(0.f, 0.f, on ? gate_beta(be_bits, PADDED && p.raw_gates) : 0.f,
                            on ? gate_log_decay(g_bits, PADDED && p.raw_gates) : 0.f);
            reinterpret_cast<uint16_t *>(smem + SM_VN2)[tb * FV_T + t] = (uint16_t)(on ? node : 0);
        }
    };
    // k and q rows of a virtual tree -> B operand tile (rows beyond the tree zero-filled): thread (r16, c16) fetches
    // 16-byte piece c16 of the rows r16, r16 + 16, r16 + 32, r16 + 48, whose node ids it is handed
    auto gather_kq = [&](int uhk, int ubase, int uT, const int (&nid)[4]) {
        const int r16 = tid >> 4, c16 = tid & 15;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int u = r16 + 16 * j;
            const bool valid = u < uT;
            const size_t off = ((size_t)(ubase + (valid ? nid[j] : 0)) * p.h_qk + uhk) * FV_D + c16 * 8;
            cp_async_16(sbase + SM_B_KQ + sw128_offset(u, c16), p.k + off, valid);
            cp_async_16(sbase + SM_B_KQ + sw128_offset(FV_T + u, c16), p.q + off, valid);
        }
        cp_async_arrive_on(mbar_kq);
    };
    // k and q rows -> B operand tile by TMA: four 64-row x 64-column boxes (k and q, either K half), 128-byte
    // swizzled, completing on mbar_kq.  A box always spans 64 nodes: rows beyond the tree belong to the next tree
    // (or are zero past the end of the tensor); every use of them is masked further down.
    auto issue_kq = [&](int ub, int uhk, int ubase, int uT) {
        (void)ub; (void)uT;
        if (warp == W_TMA && elect_one()) {
            mbar_expect_tx(mbar_kq, 32768);
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                tma_load_3d(sbase + SM_B_KQ + kh * 16384, &p.tm_k, kh * 64, uhk, ubase, mbar_kq);
                tma_load_3d(sbase + SM_B_KQ + kh * 16384 + 8192, &p.tm_q, kh * 64, uhk, ubase, mbar_kq);
            }
        }
    };
    // Tree metadata of Section 3.4.2 for one tree of at most 64 nodes, built by the CTA itself one unit ahead of
    // its use: depth and root-path list (root first, node last, 0xFF beyond) of every node.  put_parent() stages
    // parent[] in shared memory (entries outside [-1, i) are reported and cut); after a CTA barrier walk_tables()
    // lets thread i climb from node i to its root, shifting each id into a 16-byte row from below, so that the
    // root ends up in byte 0.  A tree with a bad parent[] or a root path of more than max_depth nodes is flagged in
    // bad_s[tb]; the unit then runs as a tree of no nodes.
    // Node i is handled by thread FV_T + i (warps 2 and 3; warps 0 and 1 issue MMAs at the same time).
    const int tnode = tid - FV_T;
    const bool tbl_thread = tid >= FV_T && tid < 2 * FV_T;
    auto put_parent = [&](int uT, int par, int tb) -> bool {
        bool bad = false;
        if (tbl_thread) {
            int pv = -1;
            if (tnode < uT) {
                pv = par;
                if (pv < -1 || pv >= tnode) { bad = true; pv = -1; }
            }
            par_s[tnode] = (signed char)pv;
        }
        if (tid == 0) bad_s[tb] = 0;
        return bad;
    };
    auto walk_tables = [&](int uT, int tb, uint32_t g_bits, uint32_t be_bits, bool my_bad) {
        if (tbl_thread) {
            int d = 0, err = my_bad ? GDN_ERR_TREE : 0;
            uint32_t w0 = 0xFFFFFFFFu, w1 = 0xFFFFFFFFu, w2 = 0xFFFFFFFFu, w3 = 0xFFFFFFFFu;
            if (tnode < uT && !err) {
                int cur = tnode;
                while (cur >= 0) {
                    if (++d > p.max_depth) { err = GDN_ERR_DEPTH; break; }
                    w3 = __funnelshift_l(w2, w3, 8);
                    w2 = __funnelshift_l(w1, w2, 8);
                    w1 = __funnelshift_l(w0, w1, 8);
                    w0 = (w0 << 8) | (uint32_t)cur;
                    cur = par_s[cur];
                }
            }
            if (err) {
                d = 0;
                report_status(p.status_dev, err);
                bad_s[tb] = 1;
            }
            (smem + SM_DEPTH + tb * SM_TABLE_STRIDE)[tnode] = (uint8_t)d;
            *reinterpret_cast<uint4 *>(smem + SM_ANC + tb * SM_TABLE_STRIDE + tnode * 16) = make_uint4(w0, w1, w2, w3);
            reinterpret_cast<float4 *>(smem + SM_GAB + tb * SM_TABLE_STRIDE)[tnode] =
                make_float4(0.f, 0.f, gate_beta(be_bits, PADDED && p.raw_gates), gate_log_decay(g_bits, PADDED && p.raw_gates));
        }
    };
    // the same two steps with the loads issued on the spot (first unit of a CTA, and behind a skipped unit)
    auto load_parent = [&](int upar, int uT, int tb) -> bool {
        return put_parent(uT, tbl_thread && tnode < uT ? p.parent[upar + tnode] : -1, tb);
    };
    auto load_tables = [&](int uh, int ubase, int uT, int tb, bool my_bad) {
        uint32_t gb = 0, bb = 0;
        if (tbl_thread && tnode < uT) {
            const size_t n = (size_t)(ubase + tnode);
            gb = __ldg(reinterpret_cast<const unsigned short *>(p.g) + n * p.h_v + uh);
            bb = __ldg(reinterpret_cast<const unsigned short *>(p.beta) + n * p.h_v + uh);
        }
        walk_tables(uT, tb, gb, bb, my_bad);
    };

    // Fused commit: the accepted path of tree `ub` in the previous step goes to path slot `ps`.  One warp
    // fetches it (lane t: entry t and that node's parent) and checks with shuffles that it is a chain from a
    // root inside the previous tree; a bad path is reported and its length stored as 0, so that this state
    // stays as it was.  Readable by the other warps after the next CTA barrier.
    auto fetch_path = [&](int ub, int ps) {
        if constexpr (FUSED) {
            if (warp == 4) {
                int *slot = reinterpret_cast<int *>(smem + SM_PATH + ps * SM_PATH_SLOT);
                int pp0, len, pb = 0, pT = 0, ppar = 0;   // len 0 leaves the state alone
                if (PADDED && p.t_pad) {
                    const int tree = tree_of(ub);
                    pp0 = tree * p.path_stride;
                    len = p.path_len[tree];
                    pb = ub * p.pt_pad;
                    pT = min(p.pn_nodes[tree], p.pt_pad);
                    ppar = tree * p.pt_pad;
                } else {
                    pp0 = p.path_offsets[ub];
                    len = p.path_offsets[ub + 1] - pp0;
                    if (len != 0) {
                        pb = p.pnode_offsets[ub];
                        pT = p.pnode_offsets[ub + 1] - pb;
                        ppar = pb;
                    }
                }
                if (len != 0) {
                    const bool shape_ok = len > 0 && len <= FV_MD && len <= p.max_depth && pT > 0 && pp0 >= 0;
                    const bool mine = shape_ok && lane < len;
                    int n = -1, parent_n = -2;
                    if (mine) {
                        n = p.path[pp0 + lane];
                        if (p.pparent && n >= 0 && n < pT) parent_n = p.pparent[ppar + n];
                        slot[lane] = n;
                    }
                    const int n_up = __shfl_up_sync(0xffffffffu, n, 1);
                    bool bad = false;
                    if (mine) {
                        if (n < 0 || n >= pT) bad = true;
                        else if (p.pparent) bad = parent_n != (lane ? n_up : -1);
                        else if (lane && n <= n_up) bad = true;   // without parent[] only the topological order can be checked
                    }
                    if (__any_sync(0xffffffffu, bad) || !shape_ok) {
                        if (lane == 0) report_status(p.status_dev, GDN_ERR_PATH);
                        len = 0;
                    }
                }
                if (lane == 0) {
                    slot[16] = len;
                    slot[17] = pb;
                    slot[18] = len;
                }
            }
        }
    };
    // k and v rows of that path (bf16, 256 B each) into their parking area: issued by everybody once the slot is
    // readable and the parking area is free.  Only node ids that have been range-checked are used (slot[18] =
    // length of the path as far as it has been checked when the rows are asked for).
    auto fetch_path_kv = [&](int uh, int uhk, int ps) {
        if constexpr (FUSED) {
            const int *slot = reinterpret_cast<const int *>(smem + SM_PATH + ps * SM_PATH_SLOT);
            const int len = slot[18], pb = slot[17];
            for (int idx = tid; idx < len * 32; idx += FV_THREADS) {
                const int t = idx >> 5, c16 = idx & 15;
                const size_t n = (size_t)pb + slot[t];
                if (idx & 16)
                    cp_async_16(sbase + SM_PV + t * 256 + c16 * 16, p.pv + (n * p.h_v + uh) * FV_D + c16 * 8, true);
                else
                    cp_async_16(sbase + SM_PK + t * 256 + c16 * 16, p.pk + (n * p.h_qk + uhk) * FV_D + c16 * 8, true);
            }
        }
    };
    // per-step scalars of the path, computed on the spot (first unit of a CTA, and behind a skipped unit)
    auto path_scalars_direct = [&](int uh, int ps) {
        if constexpr (FUSED) {
            const int *slot = reinterpret_cast<const int *>(smem + SM_PATH + ps * SM_PATH_SLOT);
            float4 *ab = reinterpret_cast<float4 *>(smem + SM_PATH + ps * SM_PATH_SLOT + 128);
            const int len = slot[16], pb = slot[17];
            if (tid < len) {
                float gsum = 0.f, gt = 0.f;
                const unsigned short *pg = reinterpret_cast<const unsigned short *>(p.pg);
                const unsigned short *pbe = reinterpret_cast<const unsigned short *>(p.pbeta);
                for (int t = 0; t <= tid; ++t) {
                    gt = gate_log_decay(pg[((size_t)pb + slot[t]) * p.h_v + uh], PADDED && p.raw_gates);
                    gsum += gt;
                }
                const size_t n = (size_t)pb + slot[tid];
                const float A = expf(gsum);
                ab[tid] = make_float4(A, gate_beta(pbe[n * p.h_v + uh], PADDED && p.raw_gates), expf(gt), 1.f / A);
            }
        }
    };
    // G_i = sum of g along the root path (root first), a_i = exp(G_i), for the tables in buffer `tb`
    auto path_decay = [&](int tb) {   // four threads per node, four path positions each
        float4 *gab_t = reinterpret_cast<float4 *>(smem + SM_GAB + tb * SM_TABLE_STRIDE);
        const int i = tid >> 2, s4 = tid & 3;
        const int d = (smem + SM_DEPTH + tb * SM_TABLE_STRIDE)[i];
        const uint32_t ids = *reinterpret_cast<const uint32_t *>(smem + SM_ANC + tb * SM_TABLE_STRIDE + i * FV_MD + s4 * 4);
        float G = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (s4 * 4 + e < d) G += gab_t[(ids >> (8 * e)) & 0xFFu].w;
        G += __shfl_xor_sync(0xffffffffu, G, 1);
        G += __shfl_xor_sync(0xffffffffu, G, 2);
        if (s4 == 0) {
            gab_t[i].x = G;
            gab_t[i].y = d ? __expf(G) : 0.f;
        }
    };
    // Gram = [k;q].k^T of the tile in the k/q operand area, into TMEM columns 192..255, which nothing else uses:
    // issued by one thread as soon as the tile has landed, one unit ahead of its use.
    auto issue_gram = [&](uint32_t kq_parity) {
        if (warp == W_MMA_G && elect_one()) {
            if (!mbar_wait_bounded(mbar_kq, kq_parity)) *flag = 1;
            if constexpr (GROUPED) fence_proxy_async();   // rows written by cp.async become visible to the tensor core
            tc_fence_after();
            const uint64_t b_kq = smem_desc_sw128(sbase + SM_B_KQ);
            constexpr uint32_t id = idesc_bf16(128, 64);   // B = the 64 k rows
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t adv = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
                umma_bf16(tmem + 192, b_kq + adv, b_kq + adv, id, ks > 0);
            }
            umma_commit(mbar_g);
        }
    };

    int b = 0, h = 0, hk = 0, base = 0, T = 0, par0 = 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ... and whatever is launched behind this grid with the same attribute (the next call's kernel, which itself
    // waits for this grid to complete before it reads or writes anything) may be made resident now.
    asm volatile("griddepcontrol.launch_dependents;");
    GroupX gx{0, 0, 0, 0, true}, ngx{0, 0, 0, 0, true};
    if constexpr (GROUPED) {
        // the plan kernel has counted the groups of all trees: that many records, times the heads, times the layers
        // that share the trees in the padded layout, are the units of this grid
        int n_rec = reinterpret_cast<const volatile int32_t *>(p.unit_count)[0];
        if (reinterpret_cast<const volatile int32_t *>(p.unit_count)[1] != p.plan_magic || n_rec < 0 ||
            n_rec > p.unit_capacity) {   // not a plan of this shape (never built, or built for other sizes)
            if (tid == 0) report_status(p.status_dev, GDN_ERR_WORKSPACE);
            n_rec = 0;
        }
        const int n_layers = (PADDED && p.t_pad) ? p.n_seq / p.n_trees : 1;
        n_records = n_rec > 0 ? n_rec : 1;
        n_units = n_rec > 0 ? n_rec * p.h_v * n_layers : 0;
        gstep_h = (int)gridDim.x % p.h_v;
        const int t = (int)gridDim.x / p.h_v;
        gstep_e = t % n_records;
        gstep_l = t / n_records;
    }
    Cursor ucur = cursor_at((int)blockIdx.x);
    bool cur_ok;
    if constexpr (GROUPED) {
        cur_ok = decode_g(ucur, decode_load(ucur), b, h, hk, base, T, gx);
        while (!cur_ok && (advance(ucur), ucur.u < n_units)) cur_ok = decode_g(ucur, decode_load(ucur), b, h, hk, base, T, gx);
        int t_node, t_d;
        uint4 t_row;
        lookup_tables_g(gx, T, t_node, t_d, t_row);
        uint32_t gb = 0, bb = 0;
        if (cur_ok && tbl_thread_g() && tid - FV_T < T) {
            const size_t n = (size_t)(base + t_node);
            gb = __ldg(reinterpret_cast<const unsigned short *>(p.g) + n * p.h_v + h);
            bb = __ldg(reinterpret_cast<const unsigned short *>(p.beta) + n * p.h_v + h);
        }
        if (cur_ok) put_tables_g(T, 0, t_node, t_d, t_row, gb, bb);
        __syncthreads();
        if (cur_ok) {
            path_decay(0);
            const uint16_t *vn = reinterpret_cast<const uint16_t *>(smem + SM_VN2);
            const int nid[4] = {vn[tid >> 4], vn[(tid >> 4) + 16], vn[(tid >> 4) + 32], vn[(tid >> 4) + 48]};
            gather_kq(hk, base, T, nid);
            issue_gram(0);
        }
    } else {
        cur_ok = decode(ucur, decode_load(ucur), b, h, hk, base, T, par0);
        bool par_bad = false;
        if (cur_ok) {
            issue_kq(b, hk, base, T);
            fetch_path(b, 0);
            par_bad = load_parent(par0, T, 0);
        }
        __syncthreads();
        if (cur_ok) load_tables(h, base, T, 0, par_bad);
        __syncthreads();
        if (cur_ok) {
            path_decay(0);
            fetch_path_kv(h, hk, 0);
            path_scalars_direct(h, 0);
            issue_gram(0);
        }
    }
    int done_units = 0;
#pragma unroll 1
    for (int iter = 0; ucur.u < n_units; ++iter) {
    const bool unit_ok = cur_ok;
    const uint32_t par = (uint32_t)(done_units & 1);   // every barrier completes once per processed unit
    int nb = 0, nh = 0, nhk = 0, nbase = 0, nT = 0, npar0 = 0;
    Cursor ncur = ucur;
    advance(ncur);
    bool next_ok = false;
    const DecodeRaw next_raw = decode_load(ncur);   // looked at in the middle of the unit (stage 1)
    auto decode_next = [&]() {
        if constexpr (GROUPED) {
            next_ok = decode_g(ncur, next_raw, nb, nh, nhk, nbase, nT, ngx);
            while (!next_ok && (advance(ncur), ncur.u < n_units))   // (every record is a real group: not taken)
                next_ok = decode_g(ncur, decode_load(ncur), nb, nh, nhk, nbase, nT, ngx);
        } else {
            next_ok = decode(ncur, next_raw, nb, nh, nhk, nbase, nT, npar0);
        }
    };
    float4 *gab = reinterpret_cast<float4 *>(smem + SM_GAB + (iter & 1) * SM_TABLE_STRIDE);
    uint8_t *anc_s = smem + SM_ANC + (iter & 1) * SM_TABLE_STRIDE;
    uint8_t *depth_s = smem + SM_DEPTH + (iter & 1) * SM_TABLE_STRIDE;
    if (!unit_ok) {   // nothing to compute here: only keep the pipeline fed (never taken in the grouped mode)
        decode_next();
        if constexpr (!GROUPED) {
            __syncthreads();
            bool nbad = false;
            if (next_ok) {
                issue_kq(nb, nhk, nbase, nT);
                nbad = load_parent(npar0, nT, (iter + 1) & 1);
                fetch_path(nb, (iter + 1) & 1);
            }
            __syncthreads();
            if (next_ok) load_tables(nh, nbase, nT, (iter + 1) & 1, nbad);
            __syncthreads();
            if (next_ok) {
                path_decay((iter + 1) & 1);
                fetch_path_kv(nh, nhk, (iter + 1) & 1);
                path_scalars_direct(nh, (iter + 1) & 1);
                issue_gram(par);   // no unit was processed in between: the tile's barrier phase is this one
            }
        }
        b = nb; h = nh; hk = nhk; base = nbase; T = nT; cur_ok = next_ok;
        ucur = ncur;
        continue;
    }
    // L2 warming for this CTA's next unit, in slices at phase boundaries
    auto warm_l2_state = [&](int slice) {
        if constexpr (GROUPED) {
            // the next unit's slot is known once its record has been looked at (stage 1): both halves of the tile are
            // asked for behind that; the groups of a (tree, head) are neighbours, so most of the time L2 has it already
            if (tid == 96 && slice >= 2 && next_ok) {
                const float *S = p.S0 + (size_t)(nb * p.h_v + nh) * FV_D * FV_D + (size_t)(slice - 2) * 8192;
                prefetch_l2_bulk(S, 16384);
                prefetch_l2_bulk(S + 4096, 16384);
            }
        } else {
            if (tid == 96 && ncur.u < n_units)
                prefetch_l2_bulk(p.S0 + (size_t)(ncur.b * p.h_v + ncur.h) * FV_D * FV_D + (size_t)slice * 4096, 16384);
        }
    };

    // a tree whose parent[] was rejected while its tables were built runs as a tree of no nodes: nothing of it
    // is stored (fused form: its accepted path of the previous step is committed all the same)
    if (!GROUPED && bad_s[iter & 1]) {
        T = 0;
        if (tid < FV_T) depth_s[tid] = 0;
    }
    // (1) state tile loads: a warp instruction covers four rows; the eight lanes of a row each own one
    // 16-byte bf16 piece of either K half.  Needed only after the Gram / coefficient phases.
    float4 x[4][4];   // [row i][kh*2 + half]
    // The load/store unit takes a while to accept 64 KB of requests: the tile is asked for in pieces -- a half at the
    // top and a half behind the Gram copy when the commit needs the tile right after the coefficients; a quarter at
    // the top, a quarter behind the Gram wait and a half behind the Gram copy otherwise -- so that the threads are
    // not held at the top of the unit for all of it.
    auto load_state_rows = [&](int i0, int i1) {
        const float *S = p.S0 + (size_t)(b * p.h_v + h) * FV_D * FV_D;
#pragma unroll
        for (int i = i0; i < i1; ++i) {
            const float *src = S + (size_t)(warp * 16 + i * 4 + r4) * FV_D + l8 * 8;
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) ldg_v8(src + kh * 64, x[i][kh * 2 + 0], x[i][kh * 2 + 1]);
        }
    };
    load_state_rows(0, FUSED ? 2 : 1);
    const uint16_t *vnode_s = reinterpret_cast<const uint16_t *>(smem + SM_VN2) + (iter & 1) * FV_T;
    // this tree's v rows: one TMA box into an area that stays free until the state operand is written
    if constexpr (GROUPED) {   // ... gathered row by row (rows beyond the virtual tree zero-filled)
        const int r16 = tid >> 4, c16 = tid & 15;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int u = r16 + 16 * j;
            const bool valid = u < T;
            cp_async_16(sbase + SM_VE + u * 256 + c16 * 16,
                        p.v + ((size_t)(base + (valid ? (int)vnode_s[u] : 0)) * p.h_v + h) * FV_D + c16 * 8, valid);
        }
        cp_async_arrive_on(mbar_v);
    } else if (warp == W_TMA && elect_one()) {
        mbar_expect_tx(mbar_v, FV_T * FV_D * 2);
        tma_load_3d(sbase + SM_VE, &p.tm_v, 0, h, base, mbar_v);
    }
    // fused commit: this tree's accepted path of the previous step was fetched one unit ahead
    const float4 *ab_path = reinterpret_cast<const float4 *>(smem + SM_PATH + (iter & 1) * SM_PATH_SLOT + 128);
    int path_len = 0;
    if constexpr (FUSED) path_len = reinterpret_cast<const int *>(smem + SM_PATH + (iter & 1) * SM_PATH_SLOT)[16];

    // Everything that depends only on q, k, g, beta runs now, under the latency of the state loads.  The Gram
    // block of this unit was issued one unit ahead; every thread waits for it on its own (bounded: on expiry it
    // flags the error and everybody falls through to the clean-up).
    if (!mbar_wait_bounded(mbar_g, par)) *flag = 1;
    tc_fence_after();
    __syncthreads();
    if constexpr (!FUSED) load_state_rows(1, 2);
    warm_l2_state(0);
    if (*flag == 0) {
        // k-columns of the Gram block out of tensor memory, into the (still unused) state-operand area
        {
            const int row = (warp & 3) * 32 + lane;
            const int half = warp >> 2;   // TMEM columns 192 + 32*half .. : k_j for j = 32*half ..
            const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 192 + half * 32;
            // SMALL: only rows k_0..k_31, q_0..q_31 against columns k_0..k_31 can belong to the tree
            if (!SMALL || (half == 0 && (warp & 1) == 0)) {
                uint32_t ra[32];
                GDN_TMEM_LD32(taddr, ra);
                tmem_wait_ld();
                // row r of the copy: 16 pieces of four columns, piece c stored at position c ^ (r & 15), so that the
                // 16-byte stores of a quarter-warp (eight consecutive rows, same piece) hit all the banks once
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    *reinterpret_cast<uint4 *>(gram + row * 64 + (((half * 8 + c4) ^ (row & 15)) << 2)) =
                        make_uint4(ra[4 * c4], ra[4 * c4 + 1], ra[4 * c4 + 2], ra[4 * c4 + 3]);
            }
        }
        load_state_rows(2, 4);
        tc_fence_before();
        __syncthreads();
        warm_l2_state(1);
        // X and Y for real ancestors only; the decay ratio a_i / a_j is exp(G_i - G_j)
        // (SMALL: nodes 32.. do not exist; their rows of X and Y are never looked at)
        {
            constexpr int NU = SMALL ? 2 : 4;
            float gdiff[4], gk[4], gq[4], bi[4];
            bool on[4], onx[4];
#pragma unroll
            for (int u = 0; u < NU; ++u) {
                const int idx = u * FV_THREADS + tid;
                const int i = idx >> 4, t = idx & 15;
                const int d = depth_s[i];
                on[u] = t < d;
                onx[u] = t < d - 1;
                const int j = on[u] ? anc_s[idx] : 0;
                const float4 gi = gab[i];
                gdiff[u] = gi.x - gab[j].x;
                bi[u] = gi.z;
                const int jpos = (((j >> 2) ^ (i & 15)) << 2) | (j & 3);   // rows i and 64 + i share i & 15
                gq[u] = gram[(64 + i) * 64 + jpos];   // row 64 + i: q_i
                gk[u] = gram[i * 64 + jpos];          // row i: k_i
            }
#pragma unroll
            for (int u = 0; u < NU; ++u) {
                const int idx = u * FV_THREADS + tid;
                const float dec = __expf(gdiff[u]);
                ys[idx] = on[u] ? dec * gq[u] : 0.f;
                xs[idx] = onx[u] ? bi[u] * dec * gk[u] : 0.f;
            }
        }
    }
    cp_async_wait_all();
    __syncthreads();   // X and Y complete; the Gram copy is dead and its area can take the state operand

    // (3') fused commit: replay Eq. 7 along the previous step's accepted path on the state tile while it
    // sits in registers, write it back, and let everything below verify the new tree against it.
    // Per row c (one value component): s_c <- alpha s_c + k beta (v_c - alpha k.s_c); the eight lanes that
    // share a row reduce k.s_c with three shuffles.  The path's k/v rows were fetched above.
    const bool healthy = *flag == 0;   // uniform: every write of the flag so far lies before the barrier above
    if constexpr (FUSED) {
        if (!healthy) path_len = 0;    // a wait expired: this state is left as it was
        if (path_len > 0) {
            replay_path_on_tile(x, path_len, reinterpret_cast<const uint16_t *>(smem + SM_PK),
                                reinterpret_cast<const uint16_t *>(smem + SM_PV), ab_path, warp, r4, l8);
        }
    }
    // The v rows move into registers in the orientation of the R phase (component c = TMEM lane of this
    // thread, its 32 nodes, two bf16 per register): they are about to be overwritten by the state operand.
    uint32_t vreg[16];
    {
        if (!mbar_wait_bounded(mbar_v, par)) *flag = 1;
        const uint16_t *ve = reinterpret_cast<const uint16_t *>(smem + SM_VE) + ((warp >> 2) * 32) * FV_D +
                             (warp & 3) * 32 + lane;
#pragma unroll
        for (int m = 0; m < 16; ++m)
            vreg[m] = (uint32_t)ve[(2 * m) * FV_D] | ((uint32_t)ve[(2 * m + 1) * FV_D] << 16);
    }
    __syncthreads();   // the v rows and (FUSED) the path rows sit where the state operand is about to be written

    // (4) fp32 -> bf16 hi + lo, written as the A operand.  FUSED: the committed state -- the only state write of
    // the step -- goes out from the same registers, one 32-byte store in front of each piece's conversion so
    // that the stores drain while the arithmetic runs.
    float *S_out = nullptr;
    if constexpr (FUSED) {
        if (path_len > 0) S_out = p.S_rw + (size_t)(b * p.h_v + h) * FV_D * FV_D;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = warp * 16 + i * 4 + r4;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
            if constexpr (FUSED) {
                if (S_out) stg_v8(S_out + (size_t)row * FV_D + l8 * 8 + kh * 64, x[i][kh * 2 + 0], x[i][kh * 2 + 1]);
            }
            const float4 u = x[i][kh * 2 + 0], w = x[i][kh * 2 + 1];
            const float f[8] = {u.x, u.y, u.z, u.w, w.x, w.y, w.z, w.w};
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) split_pack_bf16(f[2 * e], f[2 * e + 1], hi[e], lo[e]);
            const uint32_t off = sw128_offset(row, kh * 8 + l8);
            *reinterpret_cast<uint4 *>(smem + SM_A_HI + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4 *>(smem + SM_A_LO + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    }
    fence_proxy_async();   // generic-proxy writes of the operand become visible to the tensor core
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    warm_l2_state(2);
    // (5) P = S0.[k;q]^T (hi then lo) on the tensor core, issued before anything else; meanwhile the loads of stage 1
    // and the back-substitution below
    if (warp == W_MMA_P && elect_one()) {
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
        umma_commit(mbar_p);
    }
    // The next unit's tables and accepted path are fetched in stages, each load issued one phase before its
    // value is used, so that no global-memory latency is paid in front of a barrier.
    // stage 1: table entries of node `tid` and the path bounds (registers only)
    int t_par = -1;
    bool t_bad = false;
    unsigned short t_g = 0, t_be = 0;
    int q_pp0 = 0, q_len = 0, q_pb = 0, q_pT = 0, q_ppar = 0, q_n = -1, q_par = -2;
    unsigned short q_g = 0, q_be = 0;
    bool q_shape_ok = false, q_mine = false;
    decode_next();
    int t_node = 0, t_d = 0;                 // grouped mode: table entries of virtual index tnode, and the
    uint4 t_row = make_uint4(0u, 0u, 0u, 0u);   // node ids of the four rows this thread gathers
    int nid[4] = {0, 0, 0, 0};
    if constexpr (GROUPED) {
        if (next_ok) {
            lookup_tables_g(ngx, nT, t_node, t_d, t_row);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int u = (tid >> 4) + 16 * j;
                nid[j] = u < nT ? vnode_global(ngx, u) : 0;
            }
        }
    }
    if (!GROUPED && next_ok) {
        if (tbl_thread && tnode < nT) {
            const int n = nbase + tnode;
            t_par = __ldg(p.parent + npar0 + tnode);
            t_g = __ldg(reinterpret_cast<const unsigned short *>(p.g) + (size_t)n * p.h_v + nh);
            t_be = __ldg(reinterpret_cast<const unsigned short *>(p.beta) + (size_t)n * p.h_v + nh);
        }
        if constexpr (FUSED) {
            if (warp == 4) {
                if (PADDED && p.t_pad) {   // (stage 2 takes differences: hand it begin / end pairs)
                    const int tree = tree_of(nb);
                    q_pp0 = tree * p.path_stride;
                    q_len = q_pp0 + p.path_len[tree];
                    q_pb = nb * p.pt_pad;
                    q_pT = q_pb + min(p.pn_nodes[tree], p.pt_pad);
                    q_ppar = tree * p.pt_pad;
                } else {
                    q_pp0 = p.path_offsets[nb];
                    q_len = p.path_offsets[nb + 1];
                    q_pb = p.pnode_offsets[nb];
                    q_pT = p.pnode_offsets[nb + 1];
                    q_ppar = q_pb;
                }
            }
        }
    }

    // (6) z^T = y^T (I + X_path)^-1 by back-substitution over the root path (column-oriented: once z_l is
    // final, subtract z_l X(n_l, n_t) from every z_t, t < l).  Four threads per node, thread sq of the quad
    // owning path positions 4 sq .. 4 sq + 3; z stays in registers until the k/q tile can be overwritten.
    const int zi = tid >> 2, sq = tid & 3;
        const int d = depth_s[zi];
        const int dmax = __reduce_max_sync(0xffffffffu, d);
        const uint4 row = *reinterpret_cast<const uint4 *>(anc_s + zi * 16);
        const uint32_t idw[4] = {row.x, row.y, row.z, row.w};
        const float4 y4 = *reinterpret_cast<const float4 *>(ys + zi * FV_MD + sq * 4);
        float z[4] = {y4.x, y4.y, y4.z, y4.w};
#pragma unroll
        for (int l = FV_MD - 1; l >= 1; --l) {
            if (l < dmax) {   // warp-uniform
                const float zl = __shfl_sync(0xffffffffu, z[l & 3], (lane & ~3) | (l >> 2));
                if (l < d && sq * 4 < l) {
                    const int nl = (int)((idw[l >> 2] >> ((l & 3) * 8)) & 0xFFu);
                    const float4 x4 = *reinterpret_cast<const float4 *>(xs + nl * FV_MD + sq * 4);
                    const float xv[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (sq * 4 + e < l) z[e] = fmaf(-zl, xv[e], z[e]);
                }
            }
        }
    // stage 2: the path entries
    if constexpr (FUSED) {
        if (next_ok && warp == 4) {
            q_len -= q_pp0;
            q_pT -= q_pb;
            q_shape_ok = q_len > 0 && q_len <= FV_MD && q_len <= p.max_depth && q_pT > 0 && q_pp0 >= 0;
            q_mine = q_shape_ok && lane < q_len;
            if (q_mine) q_n = p.path[q_pp0 + lane];
        }
    }
    bool unit_done_ok = false;
    // From here to the output staging every thread waits on the barriers of the tensor core and of TMA itself;
    // an expired wait only raises the flag, which is looked at behind the next CTA barrier (uniform decision).
    if (!mbar_wait_bounded(mbar_p, par)) *flag = 1;
    tc_fence_after();
    warm_l2_state(3);

    {
        // (7) both operand tiles are dead now: z is scattered into the dense bf16 hi/lo tiles Z[i][j] (zero off
        // the root path) over the state operand
        // the k/q tile is dead: start on the next unit of this CTA (its k/q tile, its tables), to be
        // consumed after the loop comes round
        if constexpr (GROUPED) {
            if (next_ok) {
                gather_kq(nhk, nbase, nT, nid);
                if (tbl_thread && tnode < nT) {   // stage 3: the gates of the node found in stage 1
                    const size_t n = (size_t)(nbase + t_node);
                    t_g = __ldg(reinterpret_cast<const unsigned short *>(p.g) + n * p.h_v + nh);
                    t_be = __ldg(reinterpret_cast<const unsigned short *>(p.beta) + n * p.h_v + nh);
                }
            }
        }
        if (!GROUPED && next_ok) {
            issue_kq(nb, nhk, nbase, nT);
            // stage 3: parent[] of the next tree is staged for the walk behind the next CTA barrier; the parents of
            // the path entries are asked for
            t_bad = put_parent(nT, t_par, (iter + 1) & 1);
            if constexpr (FUSED) {
                if (warp == 4) {
                    // the entries are published as far as they are checked (inside the previous tree), so that
                    // their rows can be asked for behind the next barrier; whether they form a chain is decided then
                    int *slot = reinterpret_cast<int *>(smem + SM_PATH + ((iter + 1) & 1) * SM_PATH_SLOT);
                    const bool in_range = q_mine && q_n >= 0 && q_n < q_pT;
                    const bool all_in = __all_sync(0xffffffffu, !q_mine || in_range);
                    if (lane < FV_MD) slot[lane] = in_range ? q_n : 0;
                    if (lane == 0) {
                        slot[17] = q_pb;
                        slot[18] = q_shape_ok && all_in ? q_len : 0;
                    }
                    if (in_range && p.pparent) q_par = p.pparent[q_ppar + q_n];
                }
            }
        }
        {
            const int i = zi;
            const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4 *>(smem + SM_Z_HI + sw128_row_offset(i, 2 * sq)) = zero4;
            *reinterpret_cast<uint4 *>(smem + SM_Z_HI + sw128_row_offset(i, 2 * sq + 1)) = zero4;
            *reinterpret_cast<uint4 *>(smem + SM_Z_LO + sw128_row_offset(i, 2 * sq)) = zero4;
            *reinterpret_cast<uint4 *>(smem + SM_Z_LO + sw128_row_offset(i, 2 * sq + 1)) = zero4;
            __syncwarp();   // the quad's zero fill precedes the scattered stores below
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = sq * 4 + e;
                if (t < d) {
                    const int j = (int)((idw[sq] >> (e * 8)) & 0xFFu);
                    float hi, lo;
                    split_bf16(z[e], hi, lo);
                    const uint32_t off = sw128_row_offset(i, j >> 3) + (j & 7) * 2;
                    *reinterpret_cast<__nv_bfloat16 *>(smem + SM_Z_HI + off) = __float2bfloat16_rn(hi);
                    *reinterpret_cast<__nv_bfloat16 *>(smem + SM_Z_LO + off) = __float2bfloat16_rn(lo);
                }
            }
        }

        // (8) all warps: r_j[c] = beta_j (v_j[c] - a_j p^k_j[c]) for component c = TMEM lane and 32 nodes,
        // split into bf16 hi/lo and stored as the K-major A operand R^T[c][j]
        {
            const int c = (warp & 3) * 32 + lane;
            const int half = warp >> 2;
            const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
#pragma unroll 1
            for (int part = 0; part < 2; ++part) {
                const int j0 = half * 32 + part * 16;
                if (SMALL && j0 >= T) {   // no node of the tree in this 16-column piece: exact zeros for the D GEMM
                    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int oct = 0; oct < 2; ++oct) {
                        const uint32_t off = sw128_row_offset(c, half * 4 + part * 2 + oct);
                        *reinterpret_cast<uint4 *>(smem + SM_RT_HI + off) = zero4;
                        *reinterpret_cast<uint4 *>(smem + SM_RT_LO + off) = zero4;
                    }
                    continue;
                }
                uint32_t rr[16];
                GDN_TMEM_LD16(taddr + j0, rr);   // columns j0 .. j0+15: p^k of 16 nodes
                float vv[16], aj[16], bj[16];
                uint32_t vpart[8];
#pragma unroll
                for (int m = 0; m < 8; ++m) vpart[m] = part ? vreg[8 + m] : vreg[m];
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const uint32_t vw = vpart[jj >> 1];
                    vv[jj] = __uint_as_float((jj & 1) ? (vw & 0xFFFF0000u) : (vw << 16));
                    const float4 gj = gab[j0 + jj];
                    aj[jj] = gj.y;
                    bj[jj] = gj.z;
                }
                tmem_wait_ld();
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    // nodes beyond the tree hold another tree's rows: their r is forced to an exact zero
                    const float r0 = j0 + 2 * e < T ? bj[2 * e] * (vv[2 * e] - aj[2 * e] * __uint_as_float(rr[2 * e])) : 0.f;
                    const float r1 = j0 + 2 * e + 1 < T
                                         ? bj[2 * e + 1] * (vv[2 * e + 1] - aj[2 * e + 1] * __uint_as_float(rr[2 * e + 1]))
                                         : 0.f;
                    split_pack_bf16(r0, r1, hi[e], lo[e]);
                }
#pragma unroll
                for (int oct = 0; oct < 2; ++oct) {
                    const uint32_t off = sw128_row_offset(c, half * 4 + part * 2 + oct);
                    *reinterpret_cast<uint4 *>(smem + SM_RT_HI + off) = make_uint4(hi[4 * oct], hi[4 * oct + 1], hi[4 * oct + 2], hi[4 * oct + 3]);
                    *reinterpret_cast<uint4 *>(smem + SM_RT_LO + off) = make_uint4(lo[4 * oct], lo[4 * oct + 1], lo[4 * oct + 2], lo[4 * oct + 3]);
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();

        // (9) second MMA group: D[c][i] = sum_j R^T[c][j] Z[i][j] with the hi/lo cross terms
        if (warp == W_MMA_D && elect_one()) {
            constexpr uint32_t id2 = idesc_bf16(128, 64);
            const uint64_t a2[2] = {smem_desc_sw128(sbase + SM_RT_HI), smem_desc_sw128(sbase + SM_RT_LO)};
            const uint64_t b2[2] = {smem_desc_sw128(sbase + SM_Z_HI), smem_desc_sw128(sbase + SM_Z_LO)};
#pragma unroll
            for (int combo = 0; combo < 3; ++combo) {   // hi.hi, lo.hi, hi.lo; lo.lo is below 2^-18 of the result
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16(tmem + 128, a2[combo & 1] + (uint64_t)(ks * 2), b2[combo >> 1] + (uint64_t)(ks * 2), id2,
                              (combo | ks) != 0);
            }
            umma_commit(mbar_d);
        }
        // stage 4: the path is checked (a chain from a root inside the previous tree) and published; the
        // per-step scalars of its nodes are asked for
        if constexpr (FUSED) {
            if (next_ok && warp == 4) {
                int *slot = reinterpret_cast<int *>(smem + SM_PATH + ((iter + 1) & 1) * SM_PATH_SLOT);
                const int n_up = __shfl_up_sync(0xffffffffu, q_n, 1);
                bool bad = false;
                if (q_mine) {
                    if (q_n < 0 || q_n >= q_pT) bad = true;
                    else if (p.pparent) bad = q_par != (lane ? n_up : -1);
                    else if (lane && q_n <= n_up) bad = true;
                }
                if (q_len != 0 && (__any_sync(0xffffffffu, bad) || !q_shape_ok)) {
                    if (lane == 0) report_status(p.status_dev, GDN_ERR_PATH);
                    q_len = 0;
                }
                if (lane == 0) {
                    slot[16] = q_len;
                    slot[17] = q_pb;
                }
                if (lane < q_len) {
                    const size_t n = (size_t)q_pb + q_n;
                    q_g = __ldg(reinterpret_cast<const unsigned short *>(p.pg) + n * p.h_v + nh);
                    q_be = __ldg(reinterpret_cast<const unsigned short *>(p.pbeta) + n * p.h_v + nh);
                }
            }
        }

        // stage 5, while the tensor core works: the next unit's tables (depth, root paths) from the staged parent[]
        if constexpr (GROUPED) {
            if (next_ok) put_tables_g(nT, (iter + 1) & 1, t_node, t_d, t_row, t_g, t_be);
        } else {
            if (next_ok) walk_tables(nT, (iter + 1) & 1, t_g, t_be, t_bad);
        }
        if (!mbar_wait_bounded(mbar_d, par)) *flag = 1;
        tc_fence_after();

        // (10) outputs: o_i[c] = scale (a_i p^q_i[c] + D[c][i]), staged through shared memory (over the
        // dead R^T tiles) so that global memory sees 16-byte stores of whole rows
        {
            const int c = (warp & 3) * 32 + lane;
            const int half = warp >> 2;
            const uint32_t trow = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            TOut *o_s = reinterpret_cast<TOut *>(smem + SM_RT_HI);   // [64][128] TOut: 16 or 32 KB
#pragma unroll 1
            for (int part = 0; part < 2; ++part) {
                const int i0 = half * 32 + part * 16;
                if constexpr (SMALL) {
                    if (i0 >= T) continue;   // rows beyond the tree are never stored
                }
                uint32_t pp[16], dd[16];
                GDN_TMEM_LD16(trow + 64 + i0, pp);    // p^q of 16 nodes
                GDN_TMEM_LD16(trow + 128 + i0, dd);
                float ai[16];
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) ai[jj] = gab[i0 + jj].y;
                tmem_wait_ld();
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const float out = p.scale * fmaf(ai[jj], __uint_as_float(pp[jj]), __uint_as_float(dd[jj]));
                    store_from_float(o_s + (i0 + jj) * FV_D + c, out);
                }
            }
        }
        __syncthreads();
        // stage 6: the next unit's decay tables, and its path rows (published above, behind a barrier now; the area
        // they land in is free)
        if (next_ok) path_decay((iter + 1) & 1);
        if (next_ok) fetch_path_kv(nh, nhk, (iter + 1) & 1);
        if constexpr (FUSED) {   // ... and the scalars of that path (asked for a phase ago)
            if (next_ok && warp == 4) {   // lane t: decay of the path up to and including step t by a prefix sum
                const float gt = lane < q_len ? gate_log_decay(q_g, PADDED && p.raw_gates) : 0.f;
                float gsum = gt;
#pragma unroll
                for (int off = 1; off < FV_MD; off <<= 1) {
                    const float up = __shfl_up_sync(0xffffffffu, gsum, off);
                    if (lane >= off) gsum += up;
                }
                if (lane < q_len) {
                    const float A = expf(gsum);
                    reinterpret_cast<float4 *>(smem + SM_PATH + ((iter + 1) & 1) * SM_PATH_SLOT + 128)[lane] =
                        make_float4(A, gate_beta(q_be, PADDED && p.raw_gates), expf(gt), 1.f / A);
                }
            }
        }
        unit_done_ok = *flag == 0;
        if (unit_done_ok) {
            constexpr int ROW_CHUNKS = FV_D * (int)sizeof(TOut) / 16;   // 16-byte pieces per output row
            uint8_t *o = static_cast<uint8_t *>(p.o);
            for (int idx = tid; idx < T * ROW_CHUNKS; idx += FV_THREADS) {
                const int i = idx / ROW_CHUNKS, ck = idx % ROW_CHUNKS;
                const uint4 val = *reinterpret_cast<const uint4 *>(smem + SM_RT_HI + (size_t)i * FV_D * sizeof(TOut) + ck * 16);
                if constexpr (GROUPED) {   // the ancestors in front of a group belong to other groups' outputs
                    if (i >= gx.n_prefix)
                        *reinterpret_cast<uint4 *>(o + (((size_t)(base + vnode_s[i]) * p.h_v + h) * FV_D) * sizeof(TOut) + ck * 16) = val;
                } else {
                    *reinterpret_cast<uint4 *>(o + (((size_t)(base + i) * p.h_v + h) * FV_D) * sizeof(TOut) + ck * 16) = val;
                }
            }
        }
    }
    ++done_units;
    if (!unit_done_ok) break;   // a bounded wait expired: stop, report, release
    if (next_ok) issue_gram((uint32_t)(done_units & 1));   // the next unit's Gram block, as soon as its tile is there
    b = nb; h = nh; hk = nhk; base = nbase; T = nT; cur_ok = next_ok;
    gx = ngx;
    ucur = ncur;
    }   // unit loop

    if (*flag != 0 && tid == 0) report_status(p.status_dev, GDN_ERR_TIMEOUT);
    cp_async_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, FV_TMEM_COLS);
}

// Tiled TMA descriptor of a packed row tensor [n_rows][heads][128] bf16: boxes of `box_cols` x 1 head x 64 rows.
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return static_cast<EncodeTiledFn>(nullptr);
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

bool make_row_tensor_map(CUtensorMap *tm, const void *ptr, int n_rows, int heads, int box_cols, bool swizzle128)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)FV_D, (cuuint64_t)heads, (cuuint64_t)n_rows};
    const cuuint64_t strides[2] = {(cuuint64_t)FV_D * 2, (cuuint64_t)heads * FV_D * 2};   // bytes, dims 1 and 2
    const cuuint32_t box[3] = {(cuuint32_t)box_cols, 1u, (cuuint32_t)FV_T};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename TOut, bool FUSED, bool GROUPED>
cudaError_t launch_fast_typed(const gdn_shape_t &s, const VerifyFastParams &p, cudaStream_t stream)
{
    // persistent CTAs, two per SM, pipelined across units
    VerifyFastParams pt = p;
    const bool padded = p.t_pad != 0;   // the padded layout and the on-chip gate activations share an instantiation
    void (*kernel)(const VerifyFastParams);
    if constexpr (GROUPED) {
        // trees of more than 64 nodes: a unit is one ancestor-closed group of a (tree, head), taken from the plan's
        // unit list (its length is read on the device; this bound only sizes the grid); rows are gathered
        pt.n_units = p.n_units * p.groups_per_tree;
        kernel = padded ? verify_sm100_persistent_kernel<TOut, false, false, true, true>
                        : verify_sm100_persistent_kernel<TOut, false, false, false, true>;
    } else {
        // trees that fit one CTA: TMA tiles of the packed row tensors
        if (!make_row_tensor_map(&pt.tm_k, p.k, s.total_nodes, s.h_qk, 64, true) ||
            !make_row_tensor_map(&pt.tm_q, p.q, s.total_nodes, s.h_qk, 64, true) ||
            !make_row_tensor_map(&pt.tm_v, p.v, s.total_nodes, s.h_v, FV_D, false))
            return cudaErrorNotSupported;
        const bool small = s.max_tree_nodes <= 32;
        kernel = small ? verify_sm100_persistent_kernel<TOut, FUSED, true, false, false>
                       : verify_sm100_persistent_kernel<TOut, FUSED, false, false, false>;
        if (padded)
            kernel = small ? verify_sm100_persistent_kernel<TOut, FUSED, true, true, false>
                           : verify_sm100_persistent_kernel<TOut, FUSED, false, true, false>;
    }
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC);
    if (e != cudaSuccess) return e;
    const int grid = pt.n_units < p.prefetch_dist ? pt.n_units : p.prefetch_dist;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(FV_THREADS);
    cfg.dynamicSmemBytes = SM_ALLOC;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, pt);
}

VerifyFastParams make_params(const gdn_shape_t &s, const float *S0, const void *q, const void *k, const void *v,
                             const void *g, const void *beta, const int32_t *node_offsets, void *o,
                             const PlanPtrs &plan, int32_t *status_dev)
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    VerifyFastParams p{};
    p.h_qk = s.h_qk; p.h_v = s.h_v; p.n_units = s.n_seq * s.h_v; p.prefetch_dist = 2 * sms; p.scale = s.scale;
    p.S0 = S0;
    p.q = static_cast<const __nv_bfloat16 *>(q); p.k = static_cast<const __nv_bfloat16 *>(k);
    p.v = static_cast<const __nv_bfloat16 *>(v); p.g = static_cast<const __nv_bfloat16 *>(g);
    p.beta = static_cast<const __nv_bfloat16 *>(beta);
    p.node_offsets = node_offsets; p.o = o;
    p.n_seq = s.n_seq; p.total_nodes = s.total_nodes; p.max_tree_nodes = s.max_tree_nodes; p.max_depth = s.max_depth;
    p.depth = plan.depth; p.anc8 = plan.anc8; p.status_dev = status_dev;
    // upper bound of the groups of a tree (the real ones are in the plan's unit list)
    p.groups_per_tree = s.max_tree_nodes <= FV_T ? 1 : (s.max_tree_nodes + GDN_GROUP_MIN_NODES - 1) / GDN_GROUP_MIN_NODES;
    p.anc_stride = s.max_depth;
    p.anc16 = plan.anc; p.dfs_node = plan.dfs_node; p.dfs_depth = plan.dfs_depth; p.dfs_anc8 = plan.dfs_anc8;
    p.unit_list = plan.unit_list;
    p.unit_count = plan.unit_count;
    p.unit_capacity = (int)unit_list_capacity(s);
    p.plan_magic = plan_magic(s.n_seq, s.max_tree_nodes, s.max_depth);
    return p;
}

}  // namespace

// Padded layout (trees of at most 64 nodes; see VerifyFastParams): the persistent kernel with FUSED = false / true.
cudaError_t launch_verify_sm100_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, const float *S0,
                                       const void *q, const void *k, const void *v, const void *g, const void *beta,
                                       const int32_t *parent, const int32_t *n_nodes, void *o, int32_t *status_dev,
                                       cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p = make_params(s, S0, q, k, v, g, beta, nullptr, o, PlanPtrs{}, status_dev);
    p.parent = parent;
    p.t_pad = s.max_tree_nodes; p.n_trees = n_trees; p.n_nodes = n_nodes; p.raw_gates = raw_gates ? 1 : 0;
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, false, false>(s, p, stream);
    return launch_fast_typed<float, false, false>(s, p, stream);
}

cudaError_t launch_commit_verify_sm100_padded(const gdn_shape_t &s, int n_trees, bool raw_gates, float *S,
                                              int prev_t_pad, const void *k_prev, const void *v_prev,
                                              const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                              const int32_t *n_nodes_prev, const int32_t *path,
                                              const int32_t *path_len, const void *q, const void *k, const void *v,
                                              const void *g, const void *beta, const int32_t *parent,
                                              const int32_t *n_nodes, void *o, int32_t *status_dev,
                                              cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p = make_params(s, S, q, k, v, g, beta, nullptr, o, PlanPtrs{}, status_dev);
    p.parent = parent;
    p.t_pad = s.max_tree_nodes; p.n_trees = n_trees; p.n_nodes = n_nodes; p.raw_gates = raw_gates ? 1 : 0;
    p.S_rw = S;
    p.pk = static_cast<const __nv_bfloat16 *>(k_prev); p.pv = static_cast<const __nv_bfloat16 *>(v_prev);
    p.pg = static_cast<const __nv_bfloat16 *>(g_prev); p.pbeta = static_cast<const __nv_bfloat16 *>(beta_prev);
    p.pparent = parent_prev; p.path = path;
    p.pt_pad = prev_t_pad; p.pn_nodes = n_nodes_prev; p.path_len = path_len; p.path_stride = s.max_depth;
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, true, false>(s, p, stream);
    return launch_fast_typed<float, true, false>(s, p, stream);
}

cudaError_t launch_verify_sm100_planned(const gdn_shape_t &s, int n_trees, bool raw_gates, const float *S0,
                                        const void *q, const void *k, const void *v, const void *g, const void *beta,
                                        const PlanPtrs &plan, void *o, int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p = make_params(s, S0, q, k, v, g, beta, nullptr, o, plan, status_dev);
    p.t_pad = s.max_tree_nodes; p.n_trees = n_trees; p.raw_gates = raw_gates ? 1 : 0;
    gdn_shape_t ps = s;   // the shape the plan was built for: n_trees trees of t_pad rows
    ps.n_seq = n_trees;
    ps.total_nodes = n_trees * s.max_tree_nodes;
    p.unit_capacity = (int)unit_list_capacity(ps);
    p.plan_magic = plan_magic(n_trees, s.max_tree_nodes, s.max_depth);
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, false, true>(s, p, stream);
    return launch_fast_typed<float, false, true>(s, p, stream);
}

bool verify_sm100_supported(const gdn_shape_t &s)
{
    return s.d_k == FV_D && s.d_v == FV_D && s.in_dtype == GDN_BF16 && s.max_tree_nodes <= GDN_GROUPED_MAX_NODES &&
           s.max_depth <= FV_MD;
}

bool verify_sm100_single_group(const gdn_shape_t &s) { return verify_sm100_supported(s) && s.max_tree_nodes <= FV_T; }

cudaError_t launch_verify_sm100(const gdn_shape_t &s, const float *S0, const void *q, const void *k,
                                const void *v, const void *g, const void *beta, const int32_t *parent,
                                const int32_t *node_offsets, void *o, const PlanPtrs &plan,
                                int32_t *status_dev, cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p = make_params(s, S0, q, k, v, g, beta, node_offsets, o, plan, status_dev);
    p.parent = parent;
    if (!verify_sm100_single_group(s)) {
        if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, false, true>(s, p, stream);
        return launch_fast_typed<float, false, true>(s, p, stream);
    }
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, false, false>(s, p, stream);
    return launch_fast_typed<float, false, false>(s, p, stream);
}

cudaError_t launch_commit_verify_sm100(const gdn_shape_t &s, float *S, const void *k_prev, const void *v_prev,
                                       const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                                       const int32_t *node_offsets_prev, const int32_t *path,
                                       const int32_t *path_offsets, const void *q, const void *k, const void *v,
                                       const void *g, const void *beta, const int32_t *parent,
                                       const int32_t *node_offsets, void *o, int32_t *status_dev,
                                       cudaStream_t stream)
{
    if (s.n_seq == 0 || s.total_nodes == 0) return cudaSuccess;
    VerifyFastParams p = make_params(s, S, q, k, v, g, beta, node_offsets, o, PlanPtrs{}, status_dev);
    p.parent = parent;
    p.S_rw = S;
    p.pk = static_cast<const __nv_bfloat16 *>(k_prev); p.pv = static_cast<const __nv_bfloat16 *>(v_prev);
    p.pg = static_cast<const __nv_bfloat16 *>(g_prev); p.pbeta = static_cast<const __nv_bfloat16 *>(beta_prev);
    p.pparent = parent_prev; p.pnode_offsets = node_offsets_prev; p.path = path; p.path_offsets = path_offsets;
    if (s.out_dtype == GDN_BF16) return launch_fast_typed<__nv_bfloat16, true, false>(s, p, stream);
    return launch_fast_typed<float, true, false>(s, p, stream);
}


}  // namespace gdn
