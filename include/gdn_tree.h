/*
 * gdn_tree.h -- C ABI of the B200 (sm_100a) library for rollback-free tree
 * verification of Gated DeltaNet (GDN) layers in speculative decoding.
 *
 * The operations are those of Section 3.4 of "Trees from Marginals":
 * every node of a draft tree is evaluated under the gated delta rule (Eq. 7)
 * conditioned only on its ancestors, starting from the committed state S0,
 * and the per-node outputs follow Eq. 8 ("verify", which never writes the
 * state); once the accepted root path is known the state is advanced along
 * that path in place ("commit", the delayed commit of Section 3.4 and the
 * last sentence of Section 3.4.2).
 *
 * Conventions common to every entry point
 *   - Pointers marked [device] are CUDA device pointers on the current
 *     device, contiguous, row-major, 16-byte aligned; pointers marked [host]
 *     are ordinary host pointers.  The caller owns every buffer.  The library
 *     allocates no memory and keeps no state between calls.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream).  The [device] entry points never
 *     synchronise; the *_host entry points synchronise the stream before
 *     returning.
 *   - Return value: GDN_OK or a negative gdn_status decided on the host
 *     before anything is launched (nothing is launched on error).
 *     Data-dependent faults that only the device can see (a bad parent[],
 *     a root path longer than max_depth, a path that is not a root chain)
 *     are reported by writing a negative gdn_status into *status_dev with
 *     an atomic compare-and-swap from 0; the affected tree then produces no
 *     output (verify) or keeps its state unchanged (commit).  The library
 *     never clears *status_dev: zero it before a sequence of calls and read
 *     it after synchronising.  Kernels never trap and never wait unboundedly.
 *   - Tensors (N = total_nodes = node_offsets[n_seq]):
 *       S0 / S      [n_seq][h_v][d_v][d_k]  fp32   (Section 3.4.2: [H_v, d_v, d_k];
 *                                                   element [c][r] is S_{r,c} of Eq. 7)
 *       q, k        [N][h_qk][d_k]          in_dtype
 *       v           [N][h_v][d_v]           in_dtype
 *       g, beta     [N][h_v]                in_dtype   g = log(alpha) <= 0
 *       o           [N][h_v][d_v]           out_dtype
 *       parent      [N] int32   index local to the node's own tree, -1 = root,
 *                               parent[i] < i (topological numbering, Section 3.4.1)
 *       node_offsets[n_seq+1] int32, node_offsets[0] = 0 (ragged packing of trees)
 *     Value head h uses key head h / (h_v / h_qk).  L2-normalising q and k
 *     and the gate activations are the caller's business.
 */
#ifndef GDN_TREE_H_
#define GDN_TREE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum gdn_dtype { GDN_F32 = 0, GDN_BF16 = 1 };

enum gdn_status {
    GDN_OK = 0,
    GDN_ERR_NULL = -1,        /* a required pointer is NULL                                   */
    GDN_ERR_SHAPE = -2,       /* a size is out of range or inconsistent                       */
    GDN_ERR_DTYPE = -3,       /* unknown in_dtype / out_dtype                                 */
    GDN_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned                             */
    GDN_ERR_UNSUPPORTED = -5, /* valid request that this build cannot run                     */
    GDN_ERR_CUDA = -6,        /* a CUDA runtime call failed (launch, copy, attribute)         */
    GDN_ERR_TREE = -7,        /* parent[] / node_offsets[] do not describe a topological forest */
    GDN_ERR_DEPTH = -8,       /* a root path has more than max_depth nodes                    */
    GDN_ERR_PATH = -9,        /* accepted path is not a root chain of its tree, or too long   */
    GDN_ERR_WORKSPACE = -10,  /* workspace pointer missing or smaller than required           */
    GDN_ERR_TIMEOUT = -11     /* a bounded device-side wait expired                           */
};

#define GDN_MAX_HEAD_DIM 128   /* d_k, d_v <= 128                     */
#define GDN_MAX_DEPTH_CAP 64   /* max_depth <= 64 nodes on a root path */
#define GDN_MAX_TREE_NODES 4096

/* Problem description shared by all entry points. */
typedef struct gdn_shape {
    int32_t n_seq;          /* B: number of trees / state slots (a sequence, or a (sequence, layer) pair) */
    int32_t h_qk;           /* q/k heads                                                   */
    int32_t h_v;            /* v heads, a multiple of h_qk                                  */
    int32_t d_k;            /* key dim, multiple of 4, <= GDN_MAX_HEAD_DIM                  */
    int32_t d_v;            /* value dim, <= GDN_MAX_HEAD_DIM                               */
    int32_t in_dtype;       /* gdn_dtype of q, k, v, g, beta                                */
    int32_t out_dtype;      /* gdn_dtype of o                                               */
    int32_t max_depth;      /* bound on the nodes of a root path, 1..GDN_MAX_DEPTH_CAP;
                               the paper's draft trees have at most 16 (Section 6)          */
    int32_t total_nodes;    /* N = node_offsets[n_seq]                                      */
    int32_t max_tree_nodes; /* upper bound on the size of any one tree, <= GDN_MAX_TREE_NODES */
    float scale;            /* multiplies o; Eq. 8 uses 1/sqrt(d_k)                         */
} gdn_shape_t;

/* Text for a gdn_status value (static storage, never NULL). */
const char *gdn_status_string(int status);

/*
 * Bytes of device scratch gdn_tree_verify needs for this shape: tree metadata
 * of Section 3.4.2 (per node its depth and ancestor list; used for trees of
 * more than 64 nodes and by the general kernel) and the solve result
 * u~ [N][h_v][d_v] fp32 of the general kernel (the quantity "u_j - w_j^T S0"
 * that the substitution of Eq. 13 returns).  Returns 0 if the shape is invalid.
 */
size_t gdn_tree_workspace_bytes(const gdn_shape_t *shape);

/*
 * Pure host check of tree and path arrays (no CUDA call): parent[] in [-1, i),
 * node_offsets monotone from 0 to total_nodes, every tree <= max_tree_nodes,
 * every root path <= max_depth nodes, and (if path_h != NULL) every accepted
 * path a chain from a root with path_offsets monotone from 0.
 * All four arrays are [host].  path_h / path_offsets_h may both be NULL.
 */
int gdn_tree_validate_host(const gdn_shape_t *shape, const int32_t *parent_h,
                           const int32_t *node_offsets_h, const int32_t *path_h,
                           const int32_t *path_offsets_h);

/*
 * Tree verification (Section 3.4.1, Eq. 7-11): for every node i of every tree,
 *   o_i = scale * q_i^T S_i,  S_i = Eq. 7 applied over the root path of i
 * (root first, i last) starting from S0 -- evaluated in the triangular form of
 * Eq. 9-11, so no per-node state is ever materialised and S0 is only read.
 *   S0, q, k, v, g, beta, parent, node_offsets : [device], read-only
 *   o            : [device], written for every node of every valid tree
 *   workspace    : [device], >= gdn_tree_workspace_bytes(shape) bytes, 256-byte aligned;
 *                  contents after the call: the tree metadata and u~ (reused by nothing else)
 *   status_dev   : [device] one int32, see "Return value" above
 */
int gdn_tree_verify(const gdn_shape_t *shape, const float *S0, const void *q, const void *k,
                    const void *v, const void *g, const void *beta, const int32_t *parent,
                    const int32_t *node_offsets, void *o, void *workspace, size_t workspace_bytes,
                    int32_t *status_dev, void *cuda_stream);

/*
 * Padded, shape-static entry points (Section 3.4.2: dense [N, T, H, d] inputs with T the padded tree
 * size, so that every shape is independent of the tree's contents and the call can be captured once
 * in a CUDA graph and replayed for every tree; "the proposal tree is shared by every GDN layer, so its
 * verification metadata is computed once per decode step"; Table 1, stage "scalars": the write
 * strengths and log-decays are formed inside the kernel from the layer's gate inputs).
 *   shape        : n_seq = number of slots (a (sequence, layer) pair), max_tree_nodes = T = rows per
 *                  slot (<= 64), total_nodes = n_seq * T, d_k = d_v = 128, in_dtype = GDN_BF16,
 *                  max_depth <= 16; anything else returns GDN_ERR_UNSUPPORTED
 *   n_trees      : number of distinct trees; n_seq % n_trees == 0 and slot b carries tree b % n_trees
 *                  (with one sequence and 48 layers: n_trees = 1, n_seq = 48 -- the tree is given once
 *                  and each CTA derives its metadata from it on chip, no metadata kernel runs)
 *   raw_gates    : 0: g = log(alpha) and beta as for gdn_tree_verify; non-zero: `g` and `beta` hold
 *                  the raw gate inputs a, b of the layer and the kernel forms g = -softplus(a),
 *                  beta = sigmoid(b) in fp32 (the Gated DeltaNet activations; the paper does not print them)
 *   q, k         : [n_seq][T][h_qk][d_k]       v, o : [n_seq][T][h_v][d_v]       g, beta : [n_seq][T][h_v]
 *   parent       : [device] int32 [n_trees][T], entries beyond a tree's node count are ignored
 *   n_nodes      : [device] int32 [n_trees], 0 .. T; rows of `o` beyond the count are never written
 * The fused form commits, for every slot, the accepted path of its tree in the PREVIOUS step
 * (prev_t_pad rows per slot; k_prev, v_prev, g_prev, beta_prev, parent_prev [n_trees][prev_t_pad],
 * n_nodes_prev [n_trees] in the same layout; parent_prev may be NULL) and verifies the new tree against
 * the advanced state, exactly as gdn_tree_commit_verify:
 *   path         : [device] int32 [n_trees][max_depth], node ids root first
 *   path_len     : [device] int32 [n_trees], 0 .. max_depth (0 leaves the states of that tree's slots alone)
 * Everything data-dependent (tree, node counts, paths) lives in device arrays: a captured call can be
 * replayed after they have been overwritten in place.  No workspace.  Errors as for gdn_tree_verify.
 */
int gdn_tree_verify_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, const float *S0,
                           const void *q, const void *k, const void *v, const void *g, const void *beta,
                           const int32_t *parent, const int32_t *n_nodes, void *o, int32_t *status_dev,
                           void *cuda_stream);

int gdn_tree_commit_verify_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, float *S,
                                  int32_t prev_t_pad, const void *k_prev, const void *v_prev, const void *g_prev,
                                  const void *beta_prev, const int32_t *parent_prev, const int32_t *n_nodes_prev,
                                  const int32_t *path, const int32_t *path_len, const void *q, const void *k,
                                  const void *v, const void *g, const void *beta, const int32_t *parent,
                                  const int32_t *n_nodes, void *o, int32_t *status_dev, void *cuda_stream);

/*
 * Padded layout for trees of any padded size up to 1024 rows, with the tree metadata as an object of its own
 * (Section 3.4.2: the proposal tree is shared by every GDN layer, "so its verification metadata is computed
 * once per decode step"): gdn_tree_plan builds the plan of the n_trees trees once; gdn_tree_verify_planned
 * verifies any number of slots (layers) against it, in one call or in several; gdn_tree_commit_padded is the
 * delayed commit (Section 3.4) in the same layout.  Shapes, layouts, raw_gates and errors as for
 * gdn_tree_verify_padded, except that shape->max_tree_nodes = T may be anything up to 1024 (trees of more
 * than 64 nodes are verified in ancestor-closed groups of a depth-first numbering, which the plan holds).
 *   plan         : [device] >= gdn_tree_plan_bytes(shape, n_trees) bytes, 256-byte aligned; written by
 *                  gdn_tree_plan, read-only for gdn_tree_verify_planned; depends on shape->max_tree_nodes,
 *                  shape->max_depth and n_trees only (not on n_seq or the head counts), and must have been
 *                  built with the same three values: a buffer no plan was built in, or a plan built for other
 *                  values, is refused on the device (GDN_ERR_WORKSPACE in *status_dev, nothing is written)
 *   gdn_tree_plan reports a bad tree (GDN_ERR_TREE, GDN_ERR_DEPTH) through *status_dev; the slots of such a
 *   tree are skipped by gdn_tree_verify_planned (nothing of them is written).
 *   gdn_tree_commit_padded: k, v, g, beta, parent [n_trees][T] (may be NULL), n_nodes, path
 *   [n_trees][max_depth], path_len [n_trees] describe the tree whose accepted path is committed; d_k = d_v =
 *   128, bf16 inputs, max_depth <= 16, else GDN_ERR_UNSUPPORTED.  A rejected path (GDN_ERR_PATH) leaves the
 *   states of that tree's slots untouched.
 * All three are shape-static and allocate nothing: plan + commit + verify can be captured in one CUDA graph.
 */
size_t gdn_tree_plan_bytes(const gdn_shape_t *shape, int32_t n_trees);

int gdn_tree_plan(const gdn_shape_t *shape, int32_t n_trees, const int32_t *parent, const int32_t *n_nodes,
                  void *plan, size_t plan_bytes, int32_t *status_dev, void *cuda_stream);

int gdn_tree_verify_planned(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, const float *S0,
                            const void *q, const void *k, const void *v, const void *g, const void *beta,
                            const void *plan, size_t plan_bytes, void *o, int32_t *status_dev, void *cuda_stream);

int gdn_tree_commit_padded(const gdn_shape_t *shape, int32_t n_trees, int32_t raw_gates, float *S, const void *k,
                           const void *v, const void *g, const void *beta, const int32_t *parent,
                           const int32_t *n_nodes, const int32_t *path, const int32_t *path_len,
                           int32_t *status_dev, void *cuda_stream);


/*
 * Per-branch recurrent verification: the baseline that Section 3.4 describes as "sequential scans
 * along tree branches" and that Section 5.2 / Figure 5 times against the fused kernel.  For every
 * leaf of every tree the state is copied and Eq. 7 is run token by token down the leaf's root path,
 * writing o_i (Eq. 8) for each node passed; prefixes shared by several branches are recomputed
 * once per branch.  Same arguments and results as gdn_tree_verify (fp32 arithmetic on CUDA cores,
 * any d_k, d_v <= 128), but no workspace.  A branch whose parent[] chain is broken or longer than
 * max_depth reports GDN_ERR_TREE / GDN_ERR_DEPTH and writes nothing; other branches still do.
 * It is here as a comparator and as an independent GPU check of the triangular-form kernels.
 */
int gdn_tree_verify_recurrent(const gdn_shape_t *shape, const float *S0, const void *q, const void *k,
                              const void *v, const void *g, const void *beta, const int32_t *parent,
                              const int32_t *node_offsets, void *o, int32_t *status_dev, void *cuda_stream);

/*
 * Commit (Section 3.4: the state write is postponed until the accepted branch is known and
 * is then a short recurrence over that branch; Section 3.4.2, end: it is the only state
 * write of a decode step): for every tree b, S[b] <- Eq. 7 replayed over
 * path[path_offsets[b] .. path_offsets[b+1]) (local node ids, root first),
 * in place.  An empty path leaves S[b] untouched.
 *   S            : [device] in: S0, out: S_new (the only state write of a decode step)
 *   k, v, g, beta, node_offsets : [device] the same packed tensors verify read
 *   parent       : [device] or NULL; when given, each path is checked to be a
 *                  root chain (GDN_ERR_PATH in *status_dev, that tree's state unchanged)
 *   path         : [device] int32 [path_offsets[n_seq]]
 *   path_offsets : [device] int32 [n_seq+1], path_offsets[0] = 0, each length <= max_depth
 */
int gdn_tree_commit(const gdn_shape_t *shape, float *S, const void *k, const void *v, const void *g,
                    const void *beta, const int32_t *parent, const int32_t *node_offsets,
                    const int32_t *path, const int32_t *path_offsets, int32_t *status_dev,
                    void *cuda_stream);

/*
 * Commit of the previous decode step fused with the verification of the next one.  Section 3.4
 * postpones the state commit to the next decoding iteration, when the accepted branch is known;
 * this entry point does both halves of that iteration in one pass over the state:
 *     S[b] <- Eq. 7 replayed over the accepted path of the PREVIOUS tree of b   (as gdn_tree_commit)
 *     o    <- verification of the NEW tree of b against that advanced state     (as gdn_tree_verify)
 * so every state tile is read from memory once and written once per step.  The results are those
 * of gdn_tree_commit followed by gdn_tree_verify (same tolerances; on the tensor-core path it is
 * one kernel, otherwise the two kernels are launched back to back).
 *   shape        : describes the NEW tree (total_nodes, max_tree_nodes) and the common head shapes
 *   S            : [device] in: committed state before the previous step, out: state after it
 *   k_prev, v_prev, g_prev, beta_prev, parent_prev (may be NULL), node_offsets_prev :
 *                  [device] the previous step's packed tensors (in_dtype), as given to its verify
 *   path, path_offsets : [device] accepted paths in the previous trees, as for gdn_tree_commit
 *   q, k, v, g, beta, parent, node_offsets, o, workspace, workspace_bytes, status_dev :
 *                  the new tree, exactly as for gdn_tree_verify
 * A rejected path (GDN_ERR_PATH) leaves that state unchanged and the new tree is verified
 * against the unchanged state.  A rejected or empty NEW tree (GDN_ERR_TREE / GDN_ERR_DEPTH, or no
 * nodes) writes no outputs; the commit of the previous step's path happens all the same.
 */
int gdn_tree_commit_verify(const gdn_shape_t *shape, float *S, const void *k_prev, const void *v_prev,
                           const void *g_prev, const void *beta_prev, const int32_t *parent_prev,
                           const int32_t *node_offsets_prev, const int32_t *path,
                           const int32_t *path_offsets, const void *q, const void *k, const void *v,
                           const void *g, const void *beta, const int32_t *parent,
                           const int32_t *node_offsets, void *o, void *workspace, size_t workspace_bytes,
                           int32_t *status_dev, void *cuda_stream);

/*
 * Host-buffer variants: same operations with every tensor in [host] memory
 * (pinned memory makes the copies asynchronous).  Inputs are copied into
 * `dev_arena` ([device], >= gdn_tree_host_arena_bytes(shape, total_path_len) bytes, 256-byte
 * aligned), the kernels run, results are copied back and the stream is
 * synchronised.  Returns the host-side status, or the device-side status if
 * that is non-zero.  total_path_len = path_offsets[n_seq] (0 for verify).
 */
size_t gdn_tree_host_arena_bytes(const gdn_shape_t *shape, int32_t total_path_len);

int gdn_tree_verify_host(const gdn_shape_t *shape, const float *S0_h, const void *q_h,
                         const void *k_h, const void *v_h, const void *g_h, const void *beta_h,
                         const int32_t *parent_h, const int32_t *node_offsets_h, void *o_h,
                         void *dev_arena, size_t arena_bytes, void *cuda_stream);

int gdn_tree_commit_host(const gdn_shape_t *shape, float *S_h, const void *k_h, const void *v_h,
                         const void *g_h, const void *beta_h, const int32_t *parent_h,
                         const int32_t *node_offsets_h, const int32_t *path_h,
                         const int32_t *path_offsets_h, int32_t total_path_len, void *dev_arena,
                         size_t arena_bytes, void *cuda_stream);

/*
 * Host-buffer variant of gdn_tree_commit_verify: one decode iteration as Section 3.4 schedules it
 * (the commit of the previous step's accepted paths, then the verification of the new trees), with
 * the state copied to the device once and copied back once.  prev_total_nodes = number of rows of
 * the previous step's packed tensors (node_offsets_prev[n_seq]); the other arguments as for the
 * two entry points above.  `dev_arena`: [device], 256-byte aligned, at least
 * gdn_tree_commit_verify_host_arena_bytes(shape, prev_total_nodes, total_path_len) bytes.
 * S_h is written back only if total_path_len > 0 (otherwise no state changes); o_h receives the
 * outputs of the new trees.  Returns the host-side status, or the device-side status if non-zero.
 * With two or more sequences the call is pipelined: the batch is cut into up to six groups of
 * sequences, and the copies up of one group, the kernels of the group before it and the copies down
 * of the group before that run at the same time (both directions of the host link busy).  The
 * copies run on two helper streams that the library creates on first use for each device and keeps
 * (the one exception to "keeps no state"); `cuda_stream` is synchronised before returning, as for
 * the other host variants, and nothing is left in flight.  Host buffers should be pinned: with
 * pageable memory the copies are staged synchronously and nothing overlaps.
 */
size_t gdn_tree_commit_verify_host_arena_bytes(const gdn_shape_t *shape, int32_t prev_total_nodes,
                                               int32_t total_path_len);

int gdn_tree_commit_verify_host(const gdn_shape_t *shape, float *S_h, int32_t prev_total_nodes,
                                const void *k_prev_h, const void *v_prev_h, const void *g_prev_h,
                                const void *beta_prev_h, const int32_t *parent_prev_h,
                                const int32_t *node_offsets_prev_h, const int32_t *path_h,
                                const int32_t *path_offsets_h, int32_t total_path_len, const void *q_h,
                                const void *k_h, const void *v_h, const void *g_h, const void *beta_h,
                                const int32_t *parent_h, const int32_t *node_offsets_h, void *o_h,
                                void *dev_arena, size_t arena_bytes, void *cuda_stream);

/*
 * Tree verification without a caller-provided workspace, for callers that cannot allocate device
 * memory at all (a server whose own pool owns every free byte, a latency-critical loop that must
 * not hit cudaMalloc's device-wide synchronisation, a plug-in that is forbidden to allocate).
 * The paper has no counterpart of this entry point; it is a packaging variant of gdn_tree_verify.
 *
 * Same arguments, results and error reporting as gdn_tree_verify, minus `workspace`: the scratch
 * is a fixed array of GDN_STATIC_SCRATCH_BYTES inside the library image, resident on every GPU
 * that loads the library until the process exits.  The call performs no cudaMalloc / cudaFree
 * and calls no allocating routine.
 *   - Limit: gdn_tree_workspace_bytes(shape) must not exceed GDN_STATIC_SCRATCH_BYTES (about
 *     one layer of 32 value heads x 128 with a tree of up to ~250 nodes); larger problems get
 *     GDN_ERR_WORKSPACE and nothing is launched.
 *   - The first call on each device does one-time set-up with that device current: the CUDA
 *     runtime loads the library's device code (which is when the array itself comes into being),
 *     the array's device address is resolved, the kernels' shared-memory attributes are set and the
 *     driver entry point for tensor maps is looked up.  Make that first call before starting any
 *     stream capture; the calls after it do none of this.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in
 *     it (verify rewrites every part it later reads, so nothing needs clearing).  Two calls
 *     whose kernels overlap on the GPU -- different streams, or the same stream from two threads
 *     without ordering -- race on it; serialise them.
 */
#define GDN_STATIC_SCRATCH_BYTES (4u << 20)
int gdn_tree_verify_static(const gdn_shape_t *shape, const float *S0, const void *q, const void *k,
                           const void *v, const void *g, const void *beta, const int32_t *parent,
                           const int32_t *node_offsets, void *o, int32_t *status_dev,
                           void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* GDN_TREE_H_ */
