/*
 * gdn_oracle.c -- fp64 CPU oracle for GDN tree verification and commit.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA library must
 * compute; it is deliberately slow and shares no code, header, table or
 * helper with the CUDA path.  Only tests, the smoke check and the CPU
 * baseline leg of the benchmark may call it.
 *
 * What it computes (paper Section 3.4.1):
 *   - Eq. 7: S_t = alpha_t (I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T
 *            with S in R^{d_k x d_v}, alpha_t = exp(g_t).
 *   - Eq. 8: o_t = q_t^T S_t / sqrt(d_k)   (the factor is the `scale` argument).
 *   - Tree conditioning (the partial order of Section 3.4.1, Fig. 3): a node
 *     receives context only from its ancestors, so the state used for node i
 *     is S0 advanced by Eq. 7 over the root path of i, root first, node i
 *     last (the cumulative decay of the paper is inclusive of the node).
 *   - Commit (Section 3.4.2, last sentence before Table 1): Eq. 7 replayed
 *     along the accepted root path, starting from S0.
 *
 * Every node re-runs its whole root path from S0: no memoisation, no
 * blocking, no reordering.  That is the "sequential scan along tree
 * branches" that Section 3.4 calls the prior method, and it is the plain
 * definition of the result.
 *
 * Layouts (all row-major, all fp64 here; the caller widens the stored
 * bf16/fp32 values exactly):
 *   S0, S_new : [n_seq][h_v][d_v][d_k]    (Section 3.4.2: state is [H_v, d_v, d_k];
 *                                          element [c][r] is S[r][c] of Eq. 7)
 *   q, k      : [N][h_qk][d_k]            N = node_offsets[n_seq]
 *   v, o      : [N][h_v][d_v]
 *   g, beta   : [N][h_v]                  g = log(alpha) <= 0
 *   parent    : [N] index local to the node's own tree, -1 for a root
 *   node_offsets : [n_seq+1]
 *   path      : [path_offsets[n_seq]] local node ids, root first
 * Value head h reads key head h / (h_v / h_qk).
 *
 *   - Gate activations ("scalars" stage of Section 3.4.2 / Table 1, which
 *     forms the write strengths beta and the log-decays from the layer's raw
 *     gate inputs; the paper does not print the activation, the reading is
 *     the Gated DeltaNet one that the input recipe also uses):
 *         g = -softplus(a) = -log(1 + e^a),   beta = sigmoid(b) = 1 / (1 + e^-b).
 *
 * Parity pins (tests/test_oracle_pins.py): dense-matrix brute force, the
 * triangular-solve form of Eq. 9-11, the masked closed form of Eq. 12,
 * chain == sequential decoding, sibling-order invariance, hand example,
 * closed forms for beta = 0 / orthonormal keys / scalar recurrence; the
 * gate activations against their functional equations, their limits and
 * independent library routines.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define GDN_ORACLE_OK 0
#define GDN_ORACLE_BAD_TREE -1
#define GDN_ORACLE_BAD_PATH -2
#define GDN_ORACLE_NOMEM -3

/* Eq. 7 applied once, in place, on S stored as [d_v][d_k] (S[c*d_k + r] = S_{r,c}).
 * ktS is caller-provided scratch of d_v doubles. */
static void eq7_step(double *S, const double *k, const double *v, double g, double beta,
                     int d_k, int d_v, double *ktS)
{
    const double alpha = exp(g);
    for (int c = 0; c < d_v; ++c) {
        double acc = 0.0;
        for (int r = 0; r < d_k; ++r) acc += k[r] * S[(size_t)c * d_k + r]; /* (k^T S)_c */
        ktS[c] = acc;
    }
    for (int c = 0; c < d_v; ++c)
        for (int r = 0; r < d_k; ++r)
            S[(size_t)c * d_k + r] =
                alpha * (S[(size_t)c * d_k + r] - beta * k[r] * ktS[c]) + beta * k[r] * v[c];
}

/* Checks parent[i] in [-1, i) for every node of every tree. */
static int check_trees(int n_seq, const int32_t *parent, const int32_t *node_offsets)
{
    if (node_offsets[0] != 0) return GDN_ORACLE_BAD_TREE;
    for (int b = 0; b < n_seq; ++b) {
        const int32_t base = node_offsets[b], T = node_offsets[b + 1] - base;
        if (T < 0) return GDN_ORACLE_BAD_TREE;
        for (int32_t i = 0; i < T; ++i) {
            const int32_t p = parent[base + i];
            if (p < -1 || p >= i) return GDN_ORACLE_BAD_TREE;
        }
    }
    return GDN_ORACLE_OK;
}

int gdn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Verify: o[i,h,:] = scale * q_i^T S_i, S_i = Eq. 7 over the root path of i from S0.
 * first_seq / n_do let the benchmark time a bounded sample of sequences; tests pass 0 / n_seq.
 */
int gdn_oracle_verify(int n_seq, int h_qk, int h_v, int d_k, int d_v, double scale,
                      const double *S0, const double *q, const double *k, const double *v,
                      const double *g, const double *beta, const int32_t *parent,
                      const int32_t *node_offsets, double *o, int first_seq, int n_do)
{
    int rc = check_trees(n_seq, parent, node_offsets);
    if (rc) return rc;
    const int rep = h_v / h_qk;
    const size_t tile = (size_t)d_k * d_v;
    int failed = 0;
    const int units = n_do * h_v;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        const int b = first_seq + u / h_v, h = u % h_v, hk = h / rep;
        const int32_t base = node_offsets[b], T = node_offsets[b + 1] - base;
        double *S = (double *)malloc(tile * sizeof(double));
        double *ktS = (double *)malloc((size_t)d_v * sizeof(double));
        int32_t *chain = (int32_t *)malloc((size_t)(T > 0 ? T : 1) * sizeof(int32_t));
        if (!S || !ktS || !chain) {
            failed = 1;
        } else {
            for (int32_t i = 0; i < T; ++i) {
                /* root path of i: walk parents upward, then replay root first */
                int m = 0;
                for (int32_t n = i; n >= 0; n = parent[base + n]) chain[m++] = n;
                memcpy(S, S0 + ((size_t)b * h_v + h) * tile, tile * sizeof(double));
                for (int t = m - 1; t >= 0; --t) {
                    const size_t n = (size_t)base + chain[t];
                    eq7_step(S, k + (n * h_qk + hk) * d_k, v + (n * h_v + h) * d_v,
                             g[n * h_v + h], beta[n * h_v + h], d_k, d_v, ktS);
                }
                const double *qi = q + (((size_t)base + i) * h_qk + hk) * d_k;
                double *oi = o + (((size_t)base + i) * h_v + h) * d_v;
                for (int c = 0; c < d_v; ++c) {
                    double acc = 0.0;
                    for (int r = 0; r < d_k; ++r) acc += qi[r] * S[(size_t)c * d_k + r];
                    oi[c] = scale * acc; /* Eq. 8 */
                }
            }
        }
        free(S);
        free(ktS);
        free(chain);
    }
    return failed ? GDN_ORACLE_NOMEM : GDN_ORACLE_OK;
}

/*
 * Commit: S_new[b,h] = Eq. 7 replayed over path[path_offsets[b] .. path_offsets[b+1]) from S0[b,h].
 * An empty path leaves the state unchanged.  The path must start at a root and each
 * entry must be a child of the previous one.
 */
int gdn_oracle_commit(int n_seq, int h_qk, int h_v, int d_k, int d_v, const double *S0,
                      const double *k, const double *v, const double *g, const double *beta,
                      const int32_t *parent, const int32_t *node_offsets, const int32_t *path,
                      const int32_t *path_offsets, double *S_new)
{
    int rc = check_trees(n_seq, parent, node_offsets);
    if (rc) return rc;
    if (path_offsets[0] != 0) return GDN_ORACLE_BAD_PATH;
    for (int b = 0; b < n_seq; ++b) {
        const int32_t base = node_offsets[b], T = node_offsets[b + 1] - base;
        const int32_t p0 = path_offsets[b], L = path_offsets[b + 1] - p0;
        if (L < 0) return GDN_ORACLE_BAD_PATH;
        for (int32_t t = 0; t < L; ++t) {
            const int32_t n = path[p0 + t];
            if (n < 0 || n >= T) return GDN_ORACLE_BAD_PATH;
            const int32_t want = (t == 0) ? -1 : path[p0 + t - 1];
            if (parent[base + n] != want) return GDN_ORACLE_BAD_PATH;
        }
    }
    const int rep = h_v / h_qk;
    const size_t tile = (size_t)d_k * d_v;
    int failed = 0;
    const int units = n_seq * h_v;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        const int b = u / h_v, h = u % h_v, hk = h / rep;
        const int32_t base = node_offsets[b];
        const int32_t p0 = path_offsets[b], L = path_offsets[b + 1] - p0;
        double *S = S_new + ((size_t)b * h_v + h) * tile;
        double *ktS = (double *)malloc((size_t)d_v * sizeof(double));
        if (!ktS) {
            failed = 1;
        } else {
            memcpy(S, S0 + ((size_t)b * h_v + h) * tile, tile * sizeof(double));
            for (int32_t t = 0; t < L; ++t) {
                const size_t n = (size_t)base + path[p0 + t];
                eq7_step(S, k + (n * h_qk + hk) * d_k, v + (n * h_v + h) * d_v, g[n * h_v + h],
                         beta[n * h_v + h], d_k, d_v, ktS);
            }
        }
        free(ktS);
    }
    return failed ? GDN_ORACLE_NOMEM : GDN_ORACLE_OK;
}


/* Gate activations of n raw gate pairs: g = -softplus(a), beta = sigmoid(b)
 * (the "scalars" stage of Section 3.4.2).  Written in the forms that do not
 * overflow for large |x|. */
void gdn_oracle_gates(int64_t n, const double *a_raw, const double *b_raw, double *g_out, double *beta_out)
{
    for (int64_t i = 0; i < n; ++i) {
        const double a = a_raw[i], b = b_raw[i];
        const double softplus = a > 0.0 ? a + log1p(exp(-a)) : log1p(exp(a));
        g_out[i] = -softplus;
        beta_out[i] = b >= 0.0 ? 1.0 / (1.0 + exp(-b)) : exp(b) / (1.0 + exp(b));
    }
}
