/*
 * treewy_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what GDN draft-tree verify + commit must
 * compute.  Only the tests, the smoke check and the bench's CPU-baseline legs may
 * call it.  It shares no code, header, table or helper with the CUDA library and
 * must never be linked into it.
 *
 * What it does, per (sequence b, value head h), independently:
 *
 *   The gated delta rule (paper Eq. 1)
 *        S_t = alpha_t * S_prev * (I - beta_t k_t k_t^T) + beta_t v_t k_t^T ,
 *        o_t = S_t q_t
 *   is walked node by node.  S_prev is the state of the node's PARENT, or the
 *   committed state S0 when parent == -1 (the recurrence "chained along every
 *   root-to-node path", Section 3, "Verifying a draft").  Every node's state is
 *   kept (full-state snapshotting, Section 2: N+1 states per head), so the state
 *   at the accepted node is simply looked up -- no closed form, no triangular
 *   solve, no pseudo-value rewrite is used to obtain states or outputs.
 *
 *   The pseudo-value of node t is exported by its definition (Section 3, "Key
 *   rewrite"):   u_t = beta_t * (v_t - alpha_t * S_prev k_t).
 *
 *   Tree indexing (Section 3, "Verifying a draft": ancestors precede a node):
 *        depth[t]    = 0 for parent == -1, else depth[parent]+1
 *        anc_mask[t] = bit t  |  anc_mask[parent]            (ancestor-or-self)
 *        L[t,h]      = log(alpha[t,h]) + L[parent,h]          (log of the cumulative
 *                      decay g_t of Eq. 2, which includes node t's own alpha)
 *        level_order = the sequence's nodes sorted by (depth, index)
 *
 * Matrix products are written as the triple loops of their definition.  The only
 * algebra applied to Eq. 1 is associativity of  S (k k^T) = (S k) k^T.
 *
 * Malformed sequences -- a node range that is not a range inside the T packed nodes, a node count
 * outside 1..max, a parent that is not an earlier node, an accepted node outside the tree -- are
 * flagged with the library's status bits and skipped (the packed layout and these rules are the
 * library's; the paper packs nothing).
 *
 * Parity status of the functions here: all pinned (see tests/test_oracle_pins.py:
 * literal-matrix chain recurrence, beta = 0 closed form, orthonormal-key
 * overwrite, N = 1 by hand, brute-force path enumeration, fp64 closed form of
 * Eq. 2 / Eq. 3 within 1e-12).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Largest tree taken; larger sequences are flagged.  64 matches the library's main calls (one 64-bit
 * ancestor mask per node); the tests of the library's wide-tree calls raise it to 128.  Nothing in
 * the arithmetic below depends on it. */
static int32_t oracle_max_nodes = 64;

void treewy_oracle_set_max_nodes(int32_t n)
{
    oracle_max_nodes = n;
}

/* per-sequence status bits (same meaning as the library's, restated here) */
#define ORACLE_SEQ_BAD_PARENT 1
#define ORACLE_SEQ_TOO_MANY_NODES 2
#define ORACLE_SEQ_BAD_ACCEPTED 4
#define ORACLE_SEQ_BAD_OFFSETS 32 /* the sequence's node range is not a range inside 0..T */

int treewy_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* 0 when sequence b is well formed, else the status bits describing why not. */
static int check_sequence(const int32_t *node_offsets, const int32_t *parent, int32_t b, int32_t T)
{
    const int32_t lo = node_offsets[b], n = node_offsets[b + 1] - lo;
    /* packed layout (the library's; the paper packs nothing): a range that is negative, runs backwards
       or ends past the T packed nodes is malformed, and nothing of it is addressed */
    if (lo < 0 || n < 0 || (int64_t)lo + n > (int64_t)T)
        return ORACLE_SEQ_BAD_OFFSETS;
    if (n < 1 || n > oracle_max_nodes)
        return ORACLE_SEQ_TOO_MANY_NODES;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t p = parent[lo + i];
        if (p < -1 || p >= i)
            return ORACLE_SEQ_BAD_PARENT;
    }
    return 0;
}

/*
 * Tree indexing.  alpha is [T, H_v] (already widened to fp64 by the caller).
 * depth [T], anc_mask [T], L [T, H_v], level_order [T] are written for well-formed sequences and
 * left untouched for malformed ones, whose seq_status[b] gets the reason OR-ed in.
 */
int treewy_oracle_prepare(int32_t B, int32_t T, int32_t H_v, const int32_t *node_offsets,
                          const int32_t *parent, const double *alpha, int32_t *depth,
                          uint64_t *anc_mask, double *L, uint8_t *level_order,
                          int32_t *seq_status)
{
    for (int32_t b = 0; b < B; ++b) {
        const int bad = check_sequence(node_offsets, parent, b, T);
        if (bad) {
            if (seq_status)
                seq_status[b] |= bad;
            continue;
        }
        const int32_t lo = node_offsets[b], n = node_offsets[b + 1] - lo;
        for (int32_t i = 0; i < n; ++i) {
            const int32_t p = parent[lo + i];
            depth[lo + i] = (p < 0) ? 0 : depth[lo + p] + 1;
            /* (a 64-bit mask holds the first 64 local nodes; bits of later nodes do not exist) */
            anc_mask[lo + i] = ((p < 0) ? 0ull : anc_mask[lo + p]) | (i < 64 ? (1ull << i) : 0ull);
            for (int32_t h = 0; h < H_v; ++h) {
                const double up = (p < 0) ? 0.0 : L[(size_t)(lo + p) * H_v + h];
                L[(size_t)(lo + i) * H_v + h] = up + log(alpha[(size_t)(lo + i) * H_v + h]);
            }
        }
        /* nodes sorted by (depth, index): one pass per depth value, in index order */
        if (level_order) {
            int32_t out = 0;
            for (int32_t d = 0; out < n; ++d)
                for (int32_t i = 0; i < n; ++i)
                    if (depth[lo + i] == d)
                        level_order[lo + out++] = (uint8_t)i;
        }
    }
    return 0;
}

/*
 * Verify + commit by snapshotting.
 *
 *   S0       [B, H_v, d_v, d_k]   committed state, d_k contiguous
 *   q, k     [T, H_qk, d_k]       value head h reads q/k head h / (H_v / H_qk)
 *   v        [T, H_v, d_v]
 *   alpha, beta [T, H_v]
 *   accepted [B]                  local node index, -1 keeps S0
 * outputs (any may be NULL):
 *   O        [T, H_v, d_v]        o_t = S_t q_t
 *   U        [T, H_v, d_v]        pseudo-values
 *   S_commit [B, H_v, d_v, d_k]   state at the accepted node
 *   Snap     [T, H_v, d_v, d_k]   every node's state (tests only; large)
 *
 * Malformed sequences (bad parent, node count outside 1..the limit, accepted outside
 * -1..N-1) are skipped: their outputs are left untouched and seq_status[b] gets
 * the reason OR-ed in.
 */
int treewy_oracle_verify_commit(int32_t B, int32_t T, int32_t H_v, int32_t H_qk, int32_t d_k, int32_t d_v,
                                const int32_t *node_offsets, const int32_t *parent,
                                const double *S0, const double *q, const double *k,
                                const double *v, const double *alpha, const double *beta,
                                const int32_t *accepted, double *O, double *U, double *S_commit,
                                double *Snap, int32_t *seq_status)
{
    if (B < 0 || H_v < 1 || H_qk < 1 || H_v % H_qk != 0 || d_k < 1 || d_v < 1)
        return 1;
    const int32_t group = H_v / H_qk;
    const size_t state = (size_t)d_v * d_k;

    for (int32_t b = 0; b < B; ++b) {
        int bad = check_sequence(node_offsets, parent, b, T);
        if (!bad && accepted) {
            const int32_t n = node_offsets[b + 1] - node_offsets[b];
            if (accepted[b] < -1 || accepted[b] >= n)
                bad = ORACLE_SEQ_BAD_ACCEPTED;
        }
        if (bad && seq_status)
            seq_status[b] |= bad;
    }

    int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < H_v; ++h) {
            const int32_t lo = node_offsets[b], n = node_offsets[b + 1] - lo;
            if (check_sequence(node_offsets, parent, b, T))
                continue;
            if (accepted && (accepted[b] < -1 || accepted[b] >= n))
                continue;

            /* the N snapshots of this (b, h), and S k */
            double *snap = (double *)malloc((size_t)n * state * sizeof(double));
            double *Sk = (double *)malloc((size_t)d_v * sizeof(double));
            if (!snap || !Sk) {
                free(snap);
                free(Sk);
#pragma omp atomic write
                failed = 1;
                continue;
            }
            const double *S_root = S0 + ((size_t)b * H_v + h) * state;
            const int32_t hq = h / group;

            for (int32_t i = 0; i < n; ++i) {
                const int32_t t = lo + i, p = parent[t];
                const double *S_prev = (p < 0) ? S_root : snap + (size_t)p * state;
                double *S_new = snap + (size_t)i * state;
                const double *kt = k + ((size_t)t * H_qk + hq) * d_k;
                const double *qt = q + ((size_t)t * H_qk + hq) * d_k;
                const double *vt = v + ((size_t)t * H_v + h) * d_v;
                const double a = alpha[(size_t)t * H_v + h];
                const double be = beta[(size_t)t * H_v + h];

                /* S_prev k_t */
                for (int32_t r = 0; r < d_v; ++r) {
                    double acc = 0.0;
                    for (int32_t c = 0; c < d_k; ++c)
                        acc += S_prev[(size_t)r * d_k + c] * kt[c];
                    Sk[r] = acc;
                }
                /* pseudo-value, by definition */
                if (U)
                    for (int32_t r = 0; r < d_v; ++r)
                        U[((size_t)t * H_v + h) * d_v + r] = be * (vt[r] - a * Sk[r]);
                /* Eq. 1: alpha * (S_prev - beta (S_prev k) k^T) + beta v k^T */
                for (int32_t r = 0; r < d_v; ++r)
                    for (int32_t c = 0; c < d_k; ++c)
                        S_new[(size_t)r * d_k + c] =
                            a * (S_prev[(size_t)r * d_k + c] - be * Sk[r] * kt[c]) +
                            be * vt[r] * kt[c];
                /* o_t = S_t q_t */
                if (O)
                    for (int32_t r = 0; r < d_v; ++r) {
                        double acc = 0.0;
                        for (int32_t c = 0; c < d_k; ++c)
                            acc += S_new[(size_t)r * d_k + c] * qt[c];
                        O[((size_t)t * H_v + h) * d_v + r] = acc;
                    }
                if (Snap)
                    memcpy(Snap + ((size_t)t * H_v + h) * state, S_new, state * sizeof(double));
            }
            if (S_commit && accepted) {
                const int32_t a_node = accepted[b];
                const double *src = (a_node < 0) ? S_root : snap + (size_t)a_node * state;
                memcpy(S_commit + ((size_t)b * H_v + h) * state, src, state * sizeof(double));
            }
            free(snap);
            free(Sk);
        }
    }
    return failed ? 2 : 0;
}
