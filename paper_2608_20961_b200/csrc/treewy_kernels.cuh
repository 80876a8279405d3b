// Argument blocks and launchers of libtreewy's kernels (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/treewy.h"

namespace treewy {

struct VerifyArgs {
    const void *S0, *q, *k, *v;
    const float *beta;
    const int32_t *node_offsets, *parent;
    const uint64_t *anc_mask;
    const float *cum_log_gate;
    const int32_t *depth;
    const uint8_t *level_order;
    void *O;
    void *U;     // fp32, or fp16 when u_half
    int u_half;
    int32_t *seq_status;
    int B, H_v, H_qk, max_nodes;
    int T;  // packed nodes: a sequence whose node range leaves 0..T is flagged and skipped
    long long wait_cycles;  // limit of the kernel's bounded waits in SM clocks (0: the default, ~2 s)
    int skip_item;          // test hook (treewy_debug_inject): the item whose loads are never issued, or -1
    // block-pool addressing: sequence b's state is states[state_index[b]] of n_states (NULL: state b of B)
    const int32_t *state_index;
    int n_states;
    // size class of this launch: sequences with cls_lo < N_b <= cls_hi are processed, the others are
    // left to the launch of their class (N_b outside 1..max_nodes is flagged where cls_lo == 0)
    int cls_lo, cls_hi;
};

// the previous decoding round, whose accepted node the fused kernel commits before verifying
struct PrevRound {
    const float *U;
    const void *k;
    const int32_t *node_offsets, *parent;
    const uint64_t *anc_mask;
    const float *cum_log_gate;
    const int32_t *accepted;
    int max_nodes;
    int T;  // packed nodes of the previous round's trees
};

struct CommitArgs {
    void *S0;
    const void *U;  // fp32, or fp16 when u_half
    int u_half;
    const void *k;
    const int32_t *node_offsets, *parent;
    const uint64_t *anc_mask;
    const float *cum_log_gate;
    const int32_t *accepted;
    float *S_out_f32;
    int32_t *seq_status;
    int B, H_v, H_qk, max_nodes;
    void *snap_out;  // snapshot mode when not NULL: [T, H_v, 128, 128] states, one per node
    int T;
    long long wait_cycles;  // as in VerifyArgs
    const int32_t *state_index;  // as in VerifyArgs
    int n_states;
};

// What treewy_debug_inject set (process-wide test hook; all zeros / -1 unless a test called it).
struct DebugInject {
    long long wait_cycles = 0;
    int skip_item = -1;
};
DebugInject &debug_inject();

cudaError_t launch_prepare(const treewy_tree_t &t, int max_nodes, const float *alpha, bool gates_are_logs,
                           int32_t *seq_status, cudaStream_t stream);
cudaError_t launch_verify_generic(const VerifyArgs &a, treewy_dtype_t io, treewy_dtype_t od,
                                  cudaStream_t stream);
// bf16 inputs: TMA + tcgen05 kernel; T = packed node count (bounds the q/k/v tensor maps)
cudaError_t launch_verify_sm100(const VerifyArgs &a, int T, treewy_dtype_t od, cudaStream_t stream);
// commit of the previous round fused into verify (trees of up to 32 nodes in the new round)
cudaError_t launch_commit_verify_sm100(const VerifyArgs &a, const PrevRound &pv, int T, treewy_dtype_t od,
                                       cudaStream_t stream);
// bf16 inputs, trees of up to SMALL_MAX_NODES nodes (chains of a few drafts above all): one small CTA
// per (sequence, head), no role pipeline; pv != NULL commits the previous round first (fused mode,
// previous trees of up to SMALL_MAX_NODES nodes as well)
constexpr int SMALL_MAX_NODES = 8;
cudaError_t launch_verify_small(const VerifyArgs &a, const PrevRound *pv, int T, treewy_dtype_t od,
                                cudaStream_t stream);
// trees of up to TREEWY_MAX_NODES_WIDE nodes, no ancestor masks (root paths are walked through the parent array):
// prepare; verify and commit dispatch on the input type -- bf16 takes the tensor-core kernel below and the
// bulk-copy commit pipeline in its parent-walk mode (CommitArgs::anc_mask == NULL), fp32 the SIMT kernels
cudaError_t launch_prepare_wide(const treewy_tree_t &t, int max_nodes, const float *alpha, int32_t *seq_status,
                                cudaStream_t stream);
cudaError_t launch_verify_wide(const VerifyArgs &a, treewy_dtype_t io, treewy_dtype_t od, cudaStream_t stream);
// ... bf16 inputs: TMA + tcgen05 for the dense contractions; trees whose deepest path has at most
// WIDE_TC_MAX_DEPTH ancestors take its fast route (ancestor lists in shared memory)
constexpr int WIDE_TC_MAX_DEPTH = 16;
cudaError_t launch_verify_wide_tc(const VerifyArgs &a, treewy_dtype_t od, cudaStream_t stream);
cudaError_t launch_commit_wide(const CommitArgs &a, treewy_dtype_t io, cudaStream_t stream);
cudaError_t launch_commit(const CommitArgs &a, treewy_dtype_t io, cudaStream_t stream);
cudaError_t launch_commit_pipe(const CommitArgs &a, cudaStream_t stream);  // bf16 state

}  // namespace treewy
