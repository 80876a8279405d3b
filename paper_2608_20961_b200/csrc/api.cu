// C ABI of libtreewy: argument checks and kernel dispatch.  No allocation, no host
// synchronisation, no state kept between calls.
#include "treewy_kernels.cuh"

using namespace treewy;

treewy::DebugInject &treewy::debug_inject()
{
    static DebugInject d;
    return d;
}

namespace {

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }
inline bool bad_ptr(const void *p) { return p == nullptr || misaligned(p); }
inline bool bad_dtype(int d) { return d != TREEWY_F32 && d != TREEWY_BF16; }

// Checks the caller-filled part of the tree; *max_nodes receives the launch bound.
treewy_status_t check_tree(const treewy_tree_t *t, bool need_outputs, int *max_nodes)
{
    if (!t) return TREEWY_ERR_INVALID_ARG;
    if (t->B < 0 || t->T < 0 || t->H_v < 1) return TREEWY_ERR_INVALID_ARG;
    if (t->max_nodes < 0) return TREEWY_ERR_INVALID_ARG;
    if (t->max_nodes > TREEWY_MAX_NODES) return TREEWY_ERR_UNSUPPORTED;
    *max_nodes = t->max_nodes == 0 ? TREEWY_MAX_NODES : t->max_nodes;
    if (t->B == 0) return TREEWY_OK;
    if (bad_ptr(t->node_offsets)) return TREEWY_ERR_INVALID_ARG;
    if (t->T > 0 && bad_ptr(t->parent)) return TREEWY_ERR_INVALID_ARG;
    if (need_outputs && t->T > 0 &&
        (bad_ptr(t->depth) || bad_ptr(t->anc_mask) || bad_ptr(t->cum_log_gate) ||
         bad_ptr(t->level_order)))
        return TREEWY_ERR_INVALID_ARG;
    return TREEWY_OK;
}

// A state view: either the plain [B,H_v,128,128] array of the classic calls (index NULL) or a block pool.
struct StateView {
    void *states;
    const int32_t *index;
    int n_states;
};
inline StateView plain_view(const void *S0, int B) { return {const_cast<void *>(S0), nullptr, B}; }
treewy_status_t check_pool(const treewy_state_pool_t *pool, StateView *out)
{
    if (!pool) return TREEWY_ERR_INVALID_ARG;
    if (pool->n_states < 0) return TREEWY_ERR_INVALID_ARG;
    if (pool->n_states > 0 && (bad_ptr(pool->states) || bad_ptr(pool->state_index))) return TREEWY_ERR_INVALID_ARG;
    *out = {pool->states, pool->state_index, pool->n_states};
    return TREEWY_OK;
}

// Every host-side check of a verify call, and its argument block.  *run is false when the call is
// valid but has nothing to do (no sequences or no nodes).  Nothing is launched here, so a call made
// of two kernels can check both halves before it enqueues the first.
treewy_status_t verify_check(StateView sv, const void *q, const void *k, const void *v, const float *beta,
                             const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                             treewy_dtype_t o_dtype, void *O, void *U, bool u_half, int32_t *seq_status,
                             VerifyArgs *out, bool *run)
{
    const void *S0 = sv.states;
    int max_nodes = 0;
    *run = false;
    treewy_status_t st = check_tree(tree, true, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (H_qk < 1 || tree->H_v % H_qk != 0) return TREEWY_ERR_INVALID_ARG;
    if (bad_dtype(io_dtype) || bad_dtype(o_dtype)) return TREEWY_ERR_UNSUPPORTED;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0 || tree->T == 0) return TREEWY_OK;
    if (bad_ptr(S0) || bad_ptr(q) || bad_ptr(k) || bad_ptr(v) || bad_ptr(beta) || bad_ptr(O) ||
        bad_ptr(U))
        return TREEWY_ERR_INVALID_ARG;

    VerifyArgs a = {};
    a.S0 = S0, a.q = q, a.k = k, a.v = v, a.beta = beta;
    a.node_offsets = tree->node_offsets, a.parent = tree->parent;
    a.anc_mask = tree->anc_mask, a.cum_log_gate = tree->cum_log_gate;
    a.depth = tree->depth, a.level_order = tree->level_order;
    a.O = O, a.U = U, a.u_half = u_half ? 1 : 0, a.seq_status = seq_status;
    a.B = tree->B, a.H_v = tree->H_v, a.H_qk = H_qk, a.max_nodes = max_nodes, a.T = tree->T;
    a.state_index = sv.index, a.n_states = sv.n_states;
    a.cls_lo = 0, a.cls_hi = max_nodes;
    a.wait_cycles = debug_inject().wait_cycles, a.skip_item = debug_inject().skip_item;
    *out = a, *run = true;
    return TREEWY_OK;
}

treewy_status_t verify_launch(const VerifyArgs &a, bool force_generic, treewy_dtype_t io_dtype,
                              treewy_dtype_t o_dtype, void *cuda_stream)
{
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (io_dtype == TREEWY_BF16 && !force_generic)
        e = launch_verify_sm100(a, a.T, o_dtype, stream);
    else
        e = launch_verify_generic(a, io_dtype, o_dtype, stream);
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t verify_common(bool force_generic, StateView sv, const void *q, const void *k,
                              const void *v, const float *beta, const treewy_tree_t *tree,
                              int32_t H_qk, treewy_dtype_t io_dtype, treewy_dtype_t o_dtype,
                              void *O, void *U, bool u_half, int32_t *seq_status, void *cuda_stream)
{
    VerifyArgs a;
    bool run = false;
    treewy_status_t st = verify_check(sv, q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O, U, u_half, seq_status, &a, &run);
    if (st != TREEWY_OK || !run) return st;
    return verify_launch(a, force_generic, io_dtype, o_dtype, cuda_stream);
}

// The same split for commit.
treewy_status_t commit_check(StateView sv, const void *U, bool u_half, const void *k, const treewy_tree_t *tree,
                             int32_t H_qk, const int32_t *accepted, treewy_dtype_t io_dtype, float *S_out_f32,
                             int32_t *seq_status, CommitArgs *out, bool *run)
{
    void *S0 = sv.states;
    int max_nodes = 0;
    *run = false;
    treewy_status_t st = check_tree(tree, true, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (H_qk < 1 || tree->H_v % H_qk != 0) return TREEWY_ERR_INVALID_ARG;
    if (bad_dtype(io_dtype)) return TREEWY_ERR_UNSUPPORTED;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (S_out_f32 && misaligned(S_out_f32)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0) return TREEWY_OK;
    if (bad_ptr(S0) || bad_ptr(accepted)) return TREEWY_ERR_INVALID_ARG;
    if (tree->T > 0 && (bad_ptr(U) || bad_ptr(k))) return TREEWY_ERR_INVALID_ARG;

    CommitArgs a = {};
    a.S0 = S0, a.U = U, a.u_half = u_half ? 1 : 0, a.k = k;
    a.node_offsets = tree->node_offsets, a.parent = tree->parent;
    a.anc_mask = tree->anc_mask, a.cum_log_gate = tree->cum_log_gate;
    a.accepted = accepted, a.S_out_f32 = S_out_f32, a.seq_status = seq_status;
    a.B = tree->B, a.H_v = tree->H_v, a.H_qk = H_qk, a.max_nodes = max_nodes;
    a.snap_out = nullptr, a.T = tree->T;
    a.state_index = sv.index, a.n_states = sv.n_states;
    a.wait_cycles = debug_inject().wait_cycles;
    *out = a, *run = true;
    return TREEWY_OK;
}

treewy_status_t commit_common(StateView sv, const void *U, bool u_half, const void *k, const treewy_tree_t *tree,
                              int32_t H_qk, const int32_t *accepted, treewy_dtype_t io_dtype, float *S_out_f32,
                              int32_t *seq_status, void *cuda_stream)
{
    CommitArgs a;
    bool run = false;
    treewy_status_t st = commit_check(sv, U, u_half, k, tree, H_qk, accepted, io_dtype, S_out_f32, seq_status, &a, &run);
    if (st != TREEWY_OK || !run) return st;
    cudaError_t e = launch_commit(a, io_dtype, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

}  // namespace

extern "C" {

static treewy_status_t prepare_common(const treewy_tree_t *tree, const float *gates, bool gates_are_logs,
                                      int32_t *seq_status, void *cuda_stream)
{
    int max_nodes = 0;
    treewy_status_t st = check_tree(tree, true, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0) return TREEWY_OK;
    if (tree->T > 0 && bad_ptr(gates)) return TREEWY_ERR_INVALID_ARG;
    cudaError_t e = launch_prepare(*tree, max_nodes, gates, gates_are_logs, seq_status,
                                   static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t treewy_tree_prepare(const treewy_tree_t *tree, const float *alpha,
                                    int32_t *seq_status, void *cuda_stream)
{
    return prepare_common(tree, alpha, false, seq_status, cuda_stream);
}

treewy_status_t treewy_tree_prepare_log(const treewy_tree_t *tree, const float *log_alpha,
                                        int32_t *seq_status, void *cuda_stream)
{
    return prepare_common(tree, log_alpha, true, seq_status, cuda_stream);
}

treewy_status_t treewy_verify(const void *S0, const void *q, const void *k, const void *v,
                              const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                              treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O, float *U,
                              int32_t *seq_status, void *cuda_stream)
{
    return verify_common(false, plain_view(S0, tree ? tree->B : 0), q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O,
                         U, false, seq_status, cuda_stream);
}

treewy_status_t treewy_verify_generic(const void *S0, const void *q, const void *k, const void *v,
                                      const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                                      treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O,
                                      float *U, int32_t *seq_status, void *cuda_stream)
{
    return verify_common(true, plain_view(S0, tree ? tree->B : 0), q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O,
                         U, false, seq_status, cuda_stream);
}

treewy_status_t treewy_commit(void *S0, const float *U, const void *k, const treewy_tree_t *tree,
                              int32_t H_qk, const int32_t *accepted, treewy_dtype_t io_dtype,
                              float *S_out_f32, int32_t *seq_status, void *cuda_stream)
{
    return commit_common(plain_view(S0, tree ? tree->B : 0), U, false, k, tree, H_qk, accepted, io_dtype, S_out_f32,
                         seq_status, cuda_stream);
}

treewy_status_t treewy_verify_half_u(const void *S0, const void *q, const void *k, const void *v, const float *beta,
                                  const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                  treewy_dtype_t o_dtype, void *O, void *U16, int32_t *seq_status, void *cuda_stream)
{
    return verify_common(false, plain_view(S0, tree ? tree->B : 0), q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O,
                         U16, true, seq_status, cuda_stream);
}

treewy_status_t treewy_commit_half_u(void *S0, const void *U16, const void *k, const treewy_tree_t *tree, int32_t H_qk,
                                  const int32_t *accepted, treewy_dtype_t io_dtype, float *S_out_f32,
                                  int32_t *seq_status, void *cuda_stream)
{
    return commit_common(plain_view(S0, tree ? tree->B : 0), U16, true, k, tree, H_qk, accepted, io_dtype, S_out_f32,
                         seq_status, cuda_stream);
}

// the caller-filled part of a wide tree (no mask needed)
static treewy_status_t check_tree_wide(const treewy_tree_t *t, int *max_nodes)
{
    if (!t) return TREEWY_ERR_INVALID_ARG;
    if (t->B < 0 || t->T < 0 || t->H_v < 1 || t->max_nodes < 0) return TREEWY_ERR_INVALID_ARG;
    if (t->max_nodes > TREEWY_MAX_NODES_WIDE) return TREEWY_ERR_UNSUPPORTED;
    *max_nodes = t->max_nodes == 0 ? TREEWY_MAX_NODES_WIDE : t->max_nodes;
    if (t->B == 0) return TREEWY_OK;
    if (bad_ptr(t->node_offsets)) return TREEWY_ERR_INVALID_ARG;
    if (t->T > 0 && (bad_ptr(t->parent) || bad_ptr(t->depth) || bad_ptr(t->cum_log_gate) || bad_ptr(t->level_order)))
        return TREEWY_ERR_INVALID_ARG;
    return TREEWY_OK;
}

treewy_status_t treewy_tree_prepare_wide(const treewy_tree_t *tree, const float *alpha, int32_t *seq_status,
                                         void *cuda_stream)
{
    int max_nodes = 0;
    treewy_status_t st = check_tree_wide(tree, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0) return TREEWY_OK;
    if (tree->T > 0 && bad_ptr(alpha)) return TREEWY_ERR_INVALID_ARG;
    cudaError_t e = launch_prepare_wide(*tree, max_nodes, alpha, seq_status, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t treewy_verify_wide(const void *S0, const void *q, const void *k, const void *v, const float *beta,
                                   const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                   treewy_dtype_t o_dtype, void *O, float *U, int32_t *seq_status, void *cuda_stream)
{
    int max_nodes = 0;
    treewy_status_t st = check_tree_wide(tree, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (H_qk < 1 || tree->H_v % H_qk != 0) return TREEWY_ERR_INVALID_ARG;
    if (bad_dtype(io_dtype) || bad_dtype(o_dtype)) return TREEWY_ERR_UNSUPPORTED;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0 || tree->T == 0) return TREEWY_OK;
    if (bad_ptr(S0) || bad_ptr(q) || bad_ptr(k) || bad_ptr(v) || bad_ptr(beta) || bad_ptr(O) || bad_ptr(U))
        return TREEWY_ERR_INVALID_ARG;
    VerifyArgs a = {};
    a.S0 = S0, a.q = q, a.k = k, a.v = v, a.beta = beta;
    a.node_offsets = tree->node_offsets, a.parent = tree->parent;
    a.cum_log_gate = tree->cum_log_gate, a.depth = tree->depth, a.level_order = tree->level_order;
    a.O = O, a.U = U, a.u_half = 0, a.seq_status = seq_status;
    a.B = tree->B, a.H_v = tree->H_v, a.H_qk = H_qk, a.max_nodes = max_nodes, a.T = tree->T;
    a.n_states = tree->B, a.cls_lo = 0, a.cls_hi = max_nodes, a.skip_item = -1;
    cudaError_t e = launch_verify_wide(a, io_dtype, o_dtype, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t treewy_commit_wide(void *S0, const float *U, const void *k, const treewy_tree_t *tree, int32_t H_qk,
                                   const int32_t *accepted, treewy_dtype_t io_dtype, float *S_out_f32,
                                   int32_t *seq_status, void *cuda_stream)
{
    int max_nodes = 0;
    treewy_status_t st = check_tree_wide(tree, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (H_qk < 1 || tree->H_v % H_qk != 0) return TREEWY_ERR_INVALID_ARG;
    if (bad_dtype(io_dtype)) return TREEWY_ERR_UNSUPPORTED;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (S_out_f32 && misaligned(S_out_f32)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0) return TREEWY_OK;
    if (bad_ptr(S0) || bad_ptr(accepted)) return TREEWY_ERR_INVALID_ARG;
    if (tree->T > 0 && (bad_ptr(U) || bad_ptr(k))) return TREEWY_ERR_INVALID_ARG;
    CommitArgs a = {};
    a.S0 = S0, a.U = U, a.u_half = 0, a.k = k;
    a.node_offsets = tree->node_offsets, a.parent = tree->parent, a.cum_log_gate = tree->cum_log_gate;
    a.accepted = accepted, a.S_out_f32 = S_out_f32, a.seq_status = seq_status;
    a.B = tree->B, a.H_v = tree->H_v, a.H_qk = H_qk, a.max_nodes = max_nodes;
    a.T = tree->T, a.n_states = tree->B;
    cudaError_t e = launch_commit_wide(a, io_dtype, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t treewy_verify_pool(const treewy_state_pool_t *pool, const void *q, const void *k, const void *v,
                                   const float *beta, const treewy_tree_t *tree, int32_t H_qk,
                                   treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O, float *U,
                                   int32_t *seq_status, void *cuda_stream)
{
    StateView sv;
    treewy_status_t st = check_pool(pool, &sv);
    if (st != TREEWY_OK) return st;
    return verify_common(false, sv, q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O, U, false, seq_status, cuda_stream);
}

treewy_status_t treewy_commit_pool(const treewy_state_pool_t *pool, const float *U, const void *k,
                                   const treewy_tree_t *tree, int32_t H_qk, const int32_t *accepted,
                                   treewy_dtype_t io_dtype, int32_t *seq_status, void *cuda_stream)
{
    StateView sv;
    treewy_status_t st = check_pool(pool, &sv);
    if (st != TREEWY_OK) return st;
    return commit_common(sv, U, false, k, tree, H_qk, accepted, io_dtype, nullptr, seq_status, cuda_stream);
}

treewy_status_t treewy_snapshot_all(const void *S0, const float *U, const void *k, const treewy_tree_t *tree,
                                    int32_t H_qk, treewy_dtype_t io_dtype, void *Snap, int32_t *seq_status,
                                    void *cuda_stream)
{
    int max_nodes = 0;
    treewy_status_t st = check_tree(tree, true, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (H_qk < 1 || tree->H_v % H_qk != 0) return TREEWY_ERR_INVALID_ARG;
    if (io_dtype != TREEWY_BF16) return TREEWY_ERR_UNSUPPORTED;
    if (seq_status && misaligned(seq_status)) return TREEWY_ERR_INVALID_ARG;
    if (tree->B == 0 || tree->T == 0) return TREEWY_OK;
    if (bad_ptr(S0) || bad_ptr(U) || bad_ptr(k) || bad_ptr(Snap)) return TREEWY_ERR_INVALID_ARG;

    CommitArgs a = {};
    a.S0 = const_cast<void *>(S0), a.U = U, a.u_half = 0, a.k = k;
    a.node_offsets = tree->node_offsets, a.parent = tree->parent;
    a.anc_mask = tree->anc_mask, a.cum_log_gate = tree->cum_log_gate;
    a.accepted = nullptr, a.S_out_f32 = nullptr, a.seq_status = seq_status;
    a.B = tree->B, a.H_v = tree->H_v, a.H_qk = H_qk, a.max_nodes = max_nodes;
    a.snap_out = Snap, a.T = tree->T;
    a.state_index = nullptr, a.n_states = tree->B;
    cudaError_t e = launch_commit_pipe(a, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

static treewy_status_t commit_verify_common(StateView sv, const float *U_prev, const void *k_prev,
                                            const treewy_tree_t *tree_prev, const int32_t *accepted_prev,
                                            const void *q, const void *k, const void *v, const float *beta,
                                            const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                            treewy_dtype_t o_dtype, void *O, float *U, int32_t single_kernel,
                                            int32_t *seq_status, void *cuda_stream)
{
    int max_prev = 0, max_nodes = 0;
    treewy_status_t st = check_tree(tree_prev, true, &max_prev);
    if (st != TREEWY_OK) return st;
    st = check_tree(tree, true, &max_nodes);
    if (st != TREEWY_OK) return st;
    if (tree_prev->B != tree->B || tree_prev->H_v != tree->H_v) return TREEWY_ERR_INVALID_ARG;
    const bool fusable = single_kernel != 0 && io_dtype == TREEWY_BF16 && max_nodes <= 32 && tree->B > 0 && tree->T > 0 && tree_prev->T > 0;
    // every check of both halves comes before the first launch: a call that is going to fail must not
    // have committed already
    CommitArgs ca;
    VerifyArgs a;
    bool run_commit = false, run_verify = false;
    st = commit_check(sv, U_prev, false, k_prev, tree_prev, H_qk, accepted_prev, io_dtype, nullptr, seq_status, &ca,
                      &run_commit);
    if (st != TREEWY_OK) return st;
    st = verify_check(sv, q, k, v, beta, tree, H_qk, io_dtype, o_dtype, O, U, false, seq_status, &a, &run_verify);
    if (st != TREEWY_OK) return st;
    if (!fusable) {  // same result from the two stand-alone kernels
        if (run_commit) {
            cudaError_t e = launch_commit(ca, io_dtype, static_cast<cudaStream_t>(cuda_stream));
            if (e != cudaSuccess) return TREEWY_ERR_CUDA;
        }
        return run_verify ? verify_launch(a, false, io_dtype, o_dtype, cuda_stream) : TREEWY_OK;
    }
    PrevRound pv;
    pv.U = U_prev, pv.k = k_prev;
    pv.node_offsets = tree_prev->node_offsets, pv.parent = tree_prev->parent;
    pv.anc_mask = tree_prev->anc_mask, pv.cum_log_gate = tree_prev->cum_log_gate;
    pv.accepted = accepted_prev, pv.max_nodes = max_prev, pv.T = tree_prev->T;
    cudaError_t e = launch_commit_verify_sm100(a, pv, tree->T, o_dtype, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TREEWY_OK : TREEWY_ERR_CUDA;
}

treewy_status_t treewy_commit_verify(void *S0, const float *U_prev, const void *k_prev,
                                     const treewy_tree_t *tree_prev, const int32_t *accepted_prev, const void *q,
                                     const void *k, const void *v, const float *beta, const treewy_tree_t *tree,
                                     int32_t H_qk, treewy_dtype_t io_dtype, treewy_dtype_t o_dtype, void *O,
                                     float *U, int32_t single_kernel, int32_t *seq_status, void *cuda_stream)
{
    return commit_verify_common(plain_view(S0, tree ? tree->B : 0), U_prev, k_prev, tree_prev, accepted_prev, q, k, v,
                                beta, tree, H_qk, io_dtype, o_dtype, O, U, single_kernel, seq_status, cuda_stream);
}

treewy_status_t treewy_commit_verify_pool(const treewy_state_pool_t *pool, const float *U_prev, const void *k_prev,
                                          const treewy_tree_t *tree_prev, const int32_t *accepted_prev,
                                          const void *q, const void *k, const void *v, const float *beta,
                                          const treewy_tree_t *tree, int32_t H_qk, treewy_dtype_t io_dtype,
                                          treewy_dtype_t o_dtype, void *O, float *U, int32_t single_kernel,
                                          int32_t *seq_status, void *cuda_stream)
{
    StateView sv;
    treewy_status_t st = check_pool(pool, &sv);
    if (st != TREEWY_OK) return st;
    return commit_verify_common(sv, U_prev, k_prev, tree_prev, accepted_prev, q, k, v, beta, tree, H_qk, io_dtype,
                                o_dtype, O, U, single_kernel, seq_status, cuda_stream);
}

void treewy_debug_inject(int64_t wait_cycles, int32_t skip_item)
{
    debug_inject().wait_cycles = wait_cycles > 0 ? wait_cycles : 0;
    debug_inject().skip_item = skip_item;
}

const char *treewy_status_string(treewy_status_t status)
{
    switch (status) {
    case TREEWY_OK: return "ok";
    case TREEWY_ERR_INVALID_ARG: return "invalid argument";
    case TREEWY_ERR_UNSUPPORTED: return "unsupported";
    case TREEWY_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

int treewy_version(void) { return 100; }

}  // extern "C"
