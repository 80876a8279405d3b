// treewy_tree_prepare: parent array -> depth, ancestor-or-self bitmask, level order, cumulative log-gate
// (Section 3, "Verifying a draft"; g_t of Eq. 2 as a running sum of log alpha).
//
// One CTA per (sequence, chunk of 16 value heads): the tree part is tiny and is recomputed by
// every chunk (only chunk 0 stores it), the log-gate part is what scales with H_v.  Every node walks up its own parent chain (depth steps, all nodes in
// parallel) for depth / mask; meanwhile all threads turn the sequence's alpha block into
// logf(alpha) in shared memory.  The cumulative log-gate of node i and head h is then the sum
// of logf(alpha[j,h]) over the set bits j of mask[i], in ascending j -- the same order a
// parent-first running sum would use -- so every (i,h) is independent and nothing is
// serialised along the tree.  level_order is a rank computation: node i goes to the position
// given by the number of nodes that sort before it by (depth, index).
#include "treewy_common.cuh"

namespace treewy {

constexpr int PREP_THREADS = 128;
constexpr int PREP_HCHUNK = 16;  // value heads per CTA

__global__ void __launch_bounds__(PREP_THREADS)
prepare_kernel(int B, int T, int H_v, int max_nodes, int gates_are_logs, const int32_t *__restrict__ node_offsets,
               const int32_t *__restrict__ parent, const float *__restrict__ alpha,
               int32_t *__restrict__ depth, uint64_t *__restrict__ anc_mask,
               float *__restrict__ cum_log_gate, uint8_t *__restrict__ level_order,
               int32_t *__restrict__ seq_status)
{
    __shared__ int s_bad;
    __shared__ int32_t s_parent[MAXN];
    __shared__ int32_t s_depth[MAXN];
    __shared__ uint64_t s_mask[MAXN];
    __shared__ float s_log[MAXN * PREP_HCHUNK];

    const int b = blockIdx.x;
    const int h0 = blockIdx.y * PREP_HCHUNK;
    grid_dependency_wait();
    grid_dependency_trigger();
    if (b >= B) return;
    const int lo = node_offsets[b];
    const int n = node_offsets[b + 1] - lo;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const int bad = validate_sequence(parent, lo, n, T, max_nodes, &s_bad);
    if (bad) {
        if (threadIdx.x == 0 && blockIdx.y == 0 && seq_status) atomicOr(&seq_status[b], bad);
        return;
    }

    for (int i = threadIdx.x; i < n; i += PREP_THREADS) s_parent[i] = parent[lo + i];
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += PREP_THREADS) {
        uint64_t m = 1ull << i;
        int d = 0;
        for (int p = s_parent[i]; p >= 0; p = s_parent[p]) m |= 1ull << p, ++d;  // parent[p] < p: ends
        s_depth[i] = d;
        s_mask[i] = m;
    }
    {
        const int hc = min(PREP_HCHUNK, H_v - h0);
        for (int e = threadIdx.x; e < n * hc; e += PREP_THREADS) {
            const int i = e / hc, h = e - i * hc;
            const float gate = alpha[(size_t)(lo + i) * H_v + h0 + h];
            s_log[i * PREP_HCHUNK + h] = gates_are_logs ? gate : logf(gate);
        }
        __syncthreads();  // log table and the tree walk are complete
        for (int e = threadIdx.x; e < n * hc; e += PREP_THREADS) {
            const int i = e / hc, h = e - i * hc;
            uint64_t m = s_mask[i];
            float acc = 0.f;
            while (m) {
                const int j = __ffsll((long long)m) - 1;
                m &= m - 1;
                acc += s_log[j * PREP_HCHUNK + h];
            }
            cum_log_gate[(size_t)(lo + i) * H_v + h0 + h] = acc;
        }
    }
    if (blockIdx.y != 0) return;
    for (int i = threadIdx.x; i < n; i += PREP_THREADS) {
        const int di = s_depth[i];
        depth[lo + i] = di;
        anc_mask[lo + i] = s_mask[i];
        // position of node i when the nodes are sorted by (depth, index)
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const int dj = s_depth[j];
            rank += (dj < di) || (dj == di && j < i);
        }
        level_order[lo + rank] = (uint8_t)i;
    }
}

cudaError_t launch_prepare(const treewy_tree_t &t, int max_nodes, const float *alpha, bool gates_are_logs,
                           int32_t *seq_status, cudaStream_t stream)
{
    if (t.B == 0) return cudaSuccess;
    const dim3 grid(t.B, (t.H_v + PREP_HCHUNK - 1) / PREP_HCHUNK);
    return launch_dependent(prepare_kernel, grid, dim3(PREP_THREADS), 0, stream, t.B, t.T, t.H_v, max_nodes,
                            gates_are_logs ? 1 : 0, t.node_offsets, t.parent, alpha, t.depth, t.anc_mask,
                            t.cum_log_gate, t.level_order, seq_status);
}

}  // namespace treewy
