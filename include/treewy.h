/*
 * treewy.h -- C ABI of libtreewy: speculative draft-tree verification and commit for
 * Gated DeltaNet (GDN) layers through the tree-structured WY transform of the gated
 * delta rule, as hand-written CUDA kernels for NVIDIA B200 (sm_100a).
 *
 * The method (TreeWY paper, Section 3).  A GDN head keeps a state S in R^{d_v x d_k} that
 * evolves by the gated delta rule (Eq. 1)
 *       S_t = alpha_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T ,   o_t = S_t q_t .
 * Writing it as S_t = alpha_t S_{t-1} + u_t k_t^T with the pseudo-value
 *       u_t = beta_t (v_t - alpha_t S_{t-1} k_t)                    ("Key rewrite")
 * and chaining it along every root-to-node path of a draft tree of N nodes that hang off
 * the committed state S0 gives ONE unit-lower-triangular system for all pseudo-values
 * (Eq. 2):
 *       (I + A) U = R ,   A[t,i] = beta_t (g_t/g_i) (k_t . k_i)  for i a proper ancestor of t,
 *                         R[t]   = beta_t (v_t - g_t S0 k_t) ,
 * with g_t the cumulative decay from S0 to t (the product of alpha over the root path,
 * node t included).  Every node's output reads out from the same solve,
 *       o_t = g_t S0 q_t + sum_{i ancestor-or-self of t} (g_t/g_i) (k_i . q_t) u_i ,
 * and once node a is accepted the next committed state is rebuilt (Eq. 3) as
 *       S_a = g_a S0 + sum_{i ancestor-or-self of a} (g_a/g_i) u_i k_i^T ,
 * so no per-node state snapshot is ever stored.
 *
 * Conventions for every call
 *   - d_k = d_v = 128 (both Qwen3.5 hybrids of the paper, Section 2).
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte aligned, and
 *     must stay valid until the stream has passed the call.  The library allocates
 *     nothing, frees nothing, keeps no global state and never synchronises the host:
 *     each call enqueues its kernel(s) on `cuda_stream` (a cudaStream_t passed as
 *     void*, NULL = the default stream) and returns.
 *   - Trees are packed: sequence b owns nodes node_offsets[b] .. node_offsets[b+1]-1
 *     (N_b = 1..64 of them), `parent` holds LOCAL indices, parent = -1 means the node
 *     applies directly to S0, and parent[i] < i (any topological order, DFS pre-order
 *     being one; Section 3, "Verifying a draft").  Several parent = -1 nodes are legal.
 *   - Value head h reads q/k head h / (H_v / H_qk) (adjacent value heads share one).
 *   - State layout: S0[b][h][r][c], r the d_v index, c the d_k index, c contiguous.
 *   - Host-checkable misuse returns an error code and launches nothing.
 *     Data-dependent errors never trap: the sequence is skipped (its rows of O / U, its
 *     tree outputs and its state are left untouched) and, when `seq_status` is not NULL,
 *     the reason is OR-ed into seq_status[b] (the caller zeroes the array).
 */
#ifndef TREEWY_H
#define TREEWY_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TREEWY_D 128         /* d_k = d_v */
#define TREEWY_MAX_NODES 64  /* nodes per sequence (one 64-bit ancestor mask per node) */
#define TREEWY_MAX_NODES_WIDE 128 /* ... for the *_wide calls, which use no masks */

typedef enum {
    TREEWY_OK = 0,
    TREEWY_ERR_INVALID_ARG = 1, /* NULL or misaligned pointer, negative size, H_v % H_qk != 0 */
    TREEWY_ERR_UNSUPPORTED = 2, /* unknown dtype, max_nodes > 64, dtype combination not built */
    TREEWY_ERR_CUDA = 3         /* launch failed; cudaGetLastError() still holds the reason */
} treewy_status_t;

typedef enum { TREEWY_F32 = 0, TREEWY_BF16 = 1 } treewy_dtype_t;

/* per-sequence status bits, OR-ed into seq_status[b] */
enum {
    TREEWY_SEQ_BAD_PARENT = 1,     /* some parent[i] >= i or < -1 */
    TREEWY_SEQ_TOO_MANY_NODES = 2, /* N_b outside 1..max_nodes */
    TREEWY_SEQ_BAD_ACCEPTED = 4,   /* accepted[b] outside -1..N_b-1 */
    TREEWY_SEQ_TIMEOUT = 8,        /* a bounded wait inside a kernel gave up */
    TREEWY_SEQ_BAD_STATE = 16,     /* state_index[b] outside 0..n_states-1 (block-pool calls) */
    TREEWY_SEQ_BAD_OFFSETS = 32    /* node_offsets[b] .. node_offsets[b+1] is not a range inside 0..T
                                      (negative, decreasing or past the T packed nodes of the tree) */
};

/*
 * A packed batch of draft trees.  The first block is filled by the caller; the second
 * is written by treewy_tree_prepare and read by treewy_verify / treewy_commit.
 */
typedef struct {
    int32_t B;                   /* sequences */
    int32_t T;                   /* packed nodes, = node_offsets[B] */
    int32_t H_v;                 /* value heads */
    int32_t max_nodes;           /* host-known upper bound on N_b, 1..64; 0 means 64.  Only
                                    sizes launches (a tight bound picks the faster kernel: up to
                                    8, 16, 32 or 64 nodes); a longer sequence is flagged, not run */
    const int32_t *node_offsets; /* [B+1] device, node_offsets[0] = 0 */
    const int32_t *parent;       /* [T]   device, local parent index or -1 */
    int32_t *depth;              /* [T]   device, out: 0 for parent = -1, else depth[parent]+1 */
    uint64_t *anc_mask;          /* [T]   device, out: bit j set <=> local node j is an
                                    ancestor of the node or the node itself */
    float *cum_log_gate;         /* [T,H_v] device, out: L[i,h] = sum over the root path of i,
                                    i included, of log(alpha[.,h])  (log of g_i in Eq. 2) */
    uint8_t *level_order;        /* [T]   device, out: each sequence's local node indices sorted by
                                    (depth, index).  Nodes of equal depth never depend on each
                                    other, so verify solves them side by side in this order */
} treewy_tree_t;

/*
 * Tree indexing (Section 3, "Verifying a draft"; g_t of Eq. 2).
 * Reads tree->node_offsets, tree->parent and alpha [T,H_v] (fp32, linear gates in (0,1]);
 * writes tree->depth, tree->anc_mask, tree->level_order (bit-exact, one correct value each)
 * and tree->cum_log_gate (fp32 sums of logf).  One small kernel on `cuda_stream`.
 * Malformed sequences get TREEWY_SEQ_BAD_PARENT / TREEWY_SEQ_TOO_MANY_NODES.
 * Topology is per decoding step, the log-gates per layer: call it once per layer, or reuse
 * depth / anc_mask across layers and let it rewrite only what changed.
 */
treewy_status_t treewy_tree_prepare(const treewy_tree_t *tree, const float *alpha,
                                    int32_t *seq_status, void *cuda_stream);

/*
 * The same with the gates given as logarithms, log_alpha [T,H_v] fp32 <= 0, which is how Gated
 * DeltaNet layers produce them (Eq. 1's alpha_t = exp(g_t)): cum_log_gate is the plain sum of
 * log_alpha along the root path, no logf is taken.  Everything else as treewy_tree_prepare.
 */
treewy_status_t treewy_tree_prepare_log(const treewy_tree_t *tree, const float *log_alpha,
                                        int32_t *seq_status, void *cuda_stream);

/*
 * Verify (Section 3, Eq. 2 and the read-out "from that same solve").
 *   S0   [B,H_v,128,128]  io_dtype, read only
 *   q,k  [T,H_qk,128]     io_dtype;  v [T,H_v,128] io_dtype;  beta [T,H_v] fp32
 *   tree                  prepared by treewy_tree_prepare with this layer's alpha
 *   O    [T,H_v,128]      o_dtype, out: o_t for every node (post-update state times q_t,
 *                         no 1/sqrt(d) scale and no normalisation are applied)
 *   U    [T,H_v,128]      fp32, out: the pseudo-values; keep them until commit
 * io_dtype = BF16 takes the tensor-core kernel; io_dtype = F32 takes the fp32 SIMT kernel.
 * o_dtype may be F32 or BF16 (round-to-nearest-even of the fp32 result).
 * Accuracy of the BF16 path: products of bf16 inputs are exact and accumulate in fp32; A, the
 * right-hand side and the solve are fp32; for batches of trees of 9 to 64 nodes the products
 * R^T (I+A)^-T and R^T ((I+A)^-1 P)^T run on the bf16 tensor pipe with every fp32 operand split
 * as x = bf16(x) + bf16(x - bf16(x)) and the lo.lo term dropped: at most 3 * 2^-18 of a product's
 * size, before the one rounding of O to o_dtype.  U is stored as computed (fp32).
 * Sequences flagged by prepare-time checks (repeated here) are skipped.
 */
treewy_status_t treewy_verify(const void *S0, const void *q, const void *k, const void *v,
                              const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                              treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O, float *U,
                              int32_t *seq_status, void *cuda_stream);

/*
 * Same contract as treewy_verify, always through the portable fp32 SIMT kernel (one CTA
 * per (sequence, value head), no tensor cores).  It is the path F32 inputs take and a
 * cross-check for the tensor-core kernel on BF16 inputs.
 */
treewy_status_t treewy_verify_generic(const void *S0, const void *q, const void *k, const void *v,
                                      const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                                      treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O,
                                      float *U, int32_t *seq_status, void *cuda_stream);

/*
 * Commit (Section 3, Eq. 3, "Reconstruct on commit").
 * For every sequence b with a = accepted[b] >= 0 and every value head h, in place:
 *   S0[b,h] <- g_a S0[b,h] + sum_{i ancestor-or-self of a} (g_a/g_i) u_i k_i^T
 * rounded once to io_dtype.  accepted[b] = -1 leaves the state as it is.
 *   S0        [B,H_v,128,128] io_dtype, in/out
 *   U         [T,H_v,128] fp32 from treewy_verify;  k [T,H_qk,128] io_dtype (same as verify)
 *   accepted  [B] int32, local node index or -1
 *   S_out_f32 optional [B,H_v,128,128] fp32: when not NULL the unrounded new state is ALSO
 *             written there (for accepted = -1 the old state, widened); NULL to skip
 * An accepted index outside -1..N_b-1 sets TREEWY_SEQ_BAD_ACCEPTED and skips the sequence.
 */
treewy_status_t treewy_commit(void *S0, const float *U, const void *k, const treewy_tree_t *tree,
                              int32_t H_qk, const int32_t *accepted, treewy_dtype_t io_dtype,
                              float *S_out_f32, int32_t *seq_status, void *cuda_stream);

/*
 * Block-pool addressing of the states (the paper keeps one state block per sequence and layer in
 * the serving engine's block pool, Section 4): sequence b's state is
 * states[state_index[b]], a [H_v,128,128] block of a pool of n_states blocks.  treewy_verify_pool
 * and treewy_commit_pool are treewy_verify and treewy_commit (without the fp32 copy) on such a
 * view; an index outside 0..n_states-1 flags TREEWY_SEQ_BAD_STATE and skips the sequence.  Two
 * sequences of one call must not share a block.
 */
typedef struct {
    void *states;               /* [n_states,H_v,128,128] io_dtype, device */
    const int32_t *state_index; /* [B] device */
    int32_t n_states;
} treewy_state_pool_t;

treewy_status_t treewy_verify_pool(const treewy_state_pool_t *pool, const void *q, const void *k, const void *v,
                                   const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                                   treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O, float *U,
                                   int32_t *seq_status, void *cuda_stream);
treewy_status_t treewy_commit_pool(const treewy_state_pool_t *pool, const float *U, const void *k,
                                   const treewy_tree_t *tree, int32_t H_qk, const int32_t *accepted,
                                   treewy_dtype_t io_dtype, int32_t *seq_status, void *cuda_stream);

/*
 * Commit of the previous round fused into the verify of this round (Section 3, Eq. 3 then Eq. 2;
 * the paper's Section 4 runs chains this way, and its deferred-state discussion in the ReplaySSM
 * appendix names the state write as the lever): in serving, a layer's commit of round r is always
 * followed by its verify of round r+1 on the same state, so one kernel reads the old state once,
 * applies Eq. 3 in shared memory, writes the new state once and verifies the new draft tree from it.
 * The result is that of
 *     treewy_commit(S0, U_prev, k_prev, tree_prev, H_qk, accepted_prev, io_dtype, NULL, ...);
 *     treewy_verify(S0, q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O, U, ...);
 * single_kernel = 0 issues exactly those two kernels.  single_kernel = 1 takes the fused kernel
 * when it applies (BF16 states, trees of up to 32 nodes in the new round; otherwise the two kernels
 * again): it moves 23 % fewer bytes.  Its rank-P update runs on the tensor cores with every fp32
 * factor split into two tf32 parts (2^-22 relative), so a few elements of the stored bf16 state may
 * differ from the two-kernel result by one rounding step; status words and the set of rows written
 * are identical.  When both rounds' trees have at most 8 nodes (max_nodes of both trees; the chain of
 * a few drafts the paper's Section 4 runs in production), a kernel of its own does the round with the
 * update in fp32 in the stand-alone commit's operation order: the stored state is then bit-identical
 * to the two-kernel result.
 * tree_prev / tree must describe the same B sequences and H_v heads; U_prev [T_prev,H_v,128] fp32
 * and k_prev [T_prev,H_qk,128] are the previous round's verify output and keys, accepted_prev [B]
 * its accepted nodes (-1 = nothing to commit for that sequence).  U_prev and U must not overlap.
 */
treewy_status_t treewy_commit_verify(void *S0, const float *U_prev, const void *k_prev,
                                     const treewy_tree_t *tree_prev, const int32_t *accepted_prev, const void *q,
                                     const void *k, const void *v, const float *beta, const treewy_tree_t *tree,
                                     int32_t H_qk, treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O,
                                     float *U, int32_t single_kernel, int32_t *seq_status, void *cuda_stream);
/* The same on a block pool of states (see treewy_state_pool_t). */
treewy_status_t treewy_commit_verify_pool(const treewy_state_pool_t *pool, const float *U_prev, const void *k_prev,
                                     const treewy_tree_t *tree_prev, const int32_t *accepted_prev, const void *q,
                                     const void *k, const void *v, const float *beta, const treewy_tree_t *tree,
                                     int32_t H_qk, treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O,
                                     float *U, int32_t single_kernel, int32_t *seq_status, void *cuda_stream);

/*
 * 16-bit pseudo-values (Section 3, "Verifying a draft": the stored pseudo-value matrix is what makes
 * the method's footprint 128 times smaller per node than a state; that ratio holds for U in a 16-bit
 * type beside a 16-bit state).  treewy_verify_half_u is treewy_verify with U written as IEEE fp16
 * [T,H_v,128]: every u is formed in fp32 exactly as in treewy_verify and rounded once (RNE) on the
 * store; O is computed from the unrounded values and is bit-identical to treewy_verify's.
 * treewy_commit_half_u is treewy_commit reading such a U (widened to fp32, fp32 accumulation, one
 * rounding of the state): the committed state differs from the fp32-U result by the rounding of U,
 * at most 2.3e-3 of the state's rms in any element and 2.2e-4 in relative Frobenius norm on the
 * benchmark workloads (fp16 keeps 11 significant bits; a bf16 U would alone break the parity gate of
 * the state).  Arguments, layouts, status bits and error behaviour are those of
 * treewy_verify / treewy_commit; U16 must be 16-byte aligned.  The fused and pool calls take fp32 U.
 */
treewy_status_t treewy_verify_half_u(const void *S0, const void *q, const void *k, const void *v, const float *beta,
                                     const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                     treewy_dtype_t o_dtype, void *O, void *U16, int32_t *seq_status,
                                     void *cuda_stream);
treewy_status_t treewy_commit_half_u(void *S0, const void *U16, const void *k, const treewy_tree_t *tree,
                                     int32_t H_qk, const int32_t *accepted, treewy_dtype_t io_dtype,
                                     float *S_out_f32, int32_t *seq_status, void *cuda_stream);

/*
 * Wide draft trees: 65 to TREEWY_MAX_NODES_WIDE nodes per sequence (the draft window is a serving
 * parameter, Section 4; Eq. 2 and Eq. 3 hold for any N).  The three calls below are
 * treewy_tree_prepare / treewy_verify / treewy_commit for such batches (smaller trees are accepted
 * too): the same arguments, layouts, status bits and error behaviour, with these differences:
 *   - tree->max_nodes may be up to TREEWY_MAX_NODES_WIDE (0 means that);
 *   - tree->anc_mask is neither written nor read and may be NULL (a root path is walked through the
 *     parent array instead); depth, cum_log_gate and level_order are written as usual;
 *   - BF16 inputs: the dense contractions (S0 [Q;K]^T and both Gram blocks) run on the tensor cores and the
 *     triangular system is solved level by level on the CUDA cores; a tree whose deepest root path has
 *     more than 16 ancestors is accepted and takes a slower route through the same kernel.  Commit of
 *     BF16 states is the bulk-copy pipeline of treewy_commit with the accepted path found by walking the
 *     parent array.  F32 inputs take plain fp32 SIMT kernels (one CTA per (sequence, value head)).
 *     No block-pool, fused or fp16-U variant.
 */
treewy_status_t treewy_tree_prepare_wide(const treewy_tree_t *tree, const float *alpha, int32_t *seq_status,
                                         void *cuda_stream);
treewy_status_t treewy_verify_wide(const void *S0, const void *q, const void *k, const void *v, const float *beta,
                                   const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                   treewy_dtype_t o_dtype, void *O, float *U, int32_t *seq_status, void *cuda_stream);
treewy_status_t treewy_commit_wide(void *S0, const float *U, const void *k, const treewy_tree_t *tree, int32_t H_qk,
                                   const int32_t *accepted, treewy_dtype_t io_dtype, float *S_out_f32,
                                   int32_t *seq_status, void *cuda_stream);

/*
 * Full-state snapshotting, the scheme the method replaces (Section 2, "Speculative verification:
 * where GDN blows up" and "Existing approaches" (i)): materialise the state of EVERY draft node,
 *   Snap[t,h] = g_t S0[b,h] + sum_{j ancestor-or-self of t} (g_t/g_j) u_j k_j^T      (Eq. 3 with a = t)
 * for each packed node t of sequence b, out of place (S0 is not modified).  Provided as a measured
 * comparator: it writes N states per sequence and head where commit writes one.
 *   S0 [B,H_v,128,128], k [T,H_qk,128]: BF16 only (F32 returns TREEWY_ERR_UNSUPPORTED);
 *   U [T,H_v,128] fp32 from treewy_verify;  Snap [T,H_v,128,128] bf16, out.
 * Malformed sequences are flagged and their states left untouched, as in treewy_commit.
 */
treewy_status_t treewy_snapshot_all(const void *S0, const float *U, const void *k, const treewy_tree_t *tree,
                                    int32_t H_qk, treewy_dtype_t io_dtype, void *Snap, int32_t *seq_status,
                                    void *cuda_stream);

/*
 * Test hook (the paper has no counterpart).  Every wait inside the pipelined kernels is bounded by one
 * deadline per kernel, about two seconds of SM clocks; a kernel whose wait runs out sets
 * TREEWY_SEQ_TIMEOUT on the sequence it was working on, frees what it holds and returns, and the
 * stream stays usable.  This call lets a test reach that path on purpose, without a fault:
 *   wait_cycles  limit of the bounded waits of later launches, in SM clocks (0 restores the default);
 *   skip_item    the (sequence * H_v + head) item whose loads treewy_verify's kernel for trees of
 *                9 to 64 nodes never issues, so every role runs into the limit (-1 = none).
 * Process-wide and not thread-safe: the only state the library keeps; never call it in production.
 */
void treewy_debug_inject(int64_t wait_cycles, int32_t skip_item);

/* A short constant string for a status code. */
const char *treewy_status_string(treewy_status_t status);

/* Library version, major * 10000 + minor * 100 + patch. */
int treewy_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TREEWY_H */
