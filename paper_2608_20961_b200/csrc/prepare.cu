// treewy_tree_prepare: parent array -> depth, ancestor-or-self bitmask, level order, cumulative log-gate
// (Section 3, "Verifying a draft"; g_t of Eq. 2 as a running sum of log alpha).
//
// One CTA per sequence.  Thread 0 walks the <= 64 nodes once for depth / mask (each node
// needs only its parent's values, and parents come first); meanwhile all threads turn the
// sequence's alpha block into logf(alpha) in shared memory.  The cumulative log-gate of
// node i and head h is then the sum of logf(alpha[j,h]) over the set bits j of mask[i], in
// ascending j -- the same order a parent-first running sum would use -- so every (i,h) is
// independent and the global loads are not serialised along the tree.
#include "treewy_common.cuh"

namespace treewy {

constexpr int PREP_THREADS = 128;
constexpr int PREP_HCHUNK = 64;  // value heads staged per pass

__global__ void __launch_bounds__(PREP_THREADS)
prepare_kernel(int B, int H_v, int max_nodes, const int32_t *__restrict__ node_offsets,
               const int32_t *__restrict__ parent, const float *__restrict__ alpha,
               int32_t *__restrict__ depth, uint64_t *__restrict__ anc_mask,
               float *__restrict__ cum_log_gate, uint8_t *__restrict__ level_order,
               int32_t *__restrict__ seq_status)
{
    __shared__ int s_bad;
    __shared__ int32_t s_depth[MAXN];
    __shared__ uint64_t s_mask[MAXN];
    __shared__ float s_log[MAXN * PREP_HCHUNK];

    const int b = blockIdx.x;
    if (b >= B) return;
    const int lo = node_offsets[b];
    const int n = node_offsets[b + 1] - lo;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const int bad = validate_sequence(parent, lo, n, max_nodes, &s_bad);
    if (bad) {
        if (threadIdx.x == 0 && seq_status) atomicOr(&seq_status[b], bad);
        return;
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < n; ++i) {
            const int p = parent[lo + i];
            s_depth[i] = (p < 0) ? 0 : s_depth[p] + 1;
            s_mask[i] = ((p < 0) ? 0ull : s_mask[p]) | (1ull << i);
        }
    }
    for (int h0 = 0; h0 < H_v; h0 += PREP_HCHUNK) {
        const int hc = min(PREP_HCHUNK, H_v - h0);
        __syncthreads();  // previous pass done with s_log (and, first time, thread 0's walk)
        for (int e = threadIdx.x; e < n * hc; e += PREP_THREADS) {
            const int i = e / hc, h = e - i * hc;
            s_log[i * PREP_HCHUNK + h] = logf(alpha[(size_t)(lo + i) * H_v + h0 + h]);
        }
        __syncthreads();
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

cudaError_t launch_prepare(const treewy_tree_t &t, int max_nodes, const float *alpha,
                           int32_t *seq_status, cudaStream_t stream)
{
    if (t.B == 0) return cudaSuccess;
    prepare_kernel<<<t.B, PREP_THREADS, 0, stream>>>(t.B, t.H_v, max_nodes, t.node_offsets,
                                                     t.parent, alpha, t.depth, t.anc_mask,
                                                     t.cum_log_gate, t.level_order, seq_status);
    return cudaGetLastError();
}

}  // namespace treewy
