// treewy_commit, bf16 production kernel (Section 3, Eq. 3):
//     S_a = g_a S0 + sum_{j ancestor-or-self of a} (g_a / g_j) u_j k_j^T ,  in place.
//
// Commit is a pure HBM stream (each 32 KiB state tile is read once and written once, with a
// handful of fp32 rank-1 terms in between), so the kernel is built around keeping bytes in
// flight rather than around threads:
//
//   * persistent grid, one CTA per SM; work item = one (sequence, value head) state tile;
//   * a ring of CP_STAGES shared-memory stages, each filled by bulk asynchronous copies (the
//     TMA engine, plain 1-D form): the contiguous 32 KiB tile plus the accepted path's k rows
//     and U rows, all counted on one mbarrier per stage;
//   * one producer warp per stage walks the short dependent chain
//     accepted -> ancestor mask / log-gate -> path log-gates, and issues the copies; four
//     producers in different phases keep that chain off the critical path;
//   * 256 consumer threads update the tile in shared memory (fp32 math, one rounding) and one
//     of them sends it back with a bulk store; the stage is handed back to its producer once
//     the store has drained the shared-memory buffer.
//
// Snapshot mode (the full-state-snapshotting comparator): the same pipeline with one item per
// (packed node, value head), the node playing the accepted node and the result going to a
// separate [T, H_v] array of states instead of back to S0.
//
// Trees of more than 64 nodes (the wide-tree calls) have no ancestor masks: there the producer warp
// keeps the sequence's parent array in shared memory and walks the accepted node's root path
// through it; everything after that is the same.
//
// Paths longer than CP_PCH nodes (deep chains) take the staged rows first and fetch the rest
// with ordinary loads.  All mbarrier waits are bounded (TREEWY_SEQ_TIMEOUT on give-up).
#include "ptx_sm100.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr int CP_STAGES = 4;
constexpr int CP_PCH = 16;  // path nodes staged per item
constexpr int CP_CONSUMERS = 256;
constexpr int CP_THREADS = CP_CONSUMERS + 32 * CP_STAGES;
constexpr uint32_t CP_TILE_BYTES = D * D * 2;
constexpr int CP_WIDE_NODES = TREEWY_MAX_NODES_WIDE;

struct __align__(128) CommitStage {
    __nv_bfloat16 tile[D * D];
    __nv_bfloat16 krow[CP_PCH][D];
    float urow[CP_PCH][D];
    float w[CP_PCH];          // e^{L_a - L_j} of the staged path nodes
    unsigned long long mask;  // ancestor-or-self mask of the accepted node
    float La, ga;             // log-gate of the accepted node and e^{La}
    int plen;                 // path length; -1 = nothing to do for this item
    int store_tile;           // 1: tile goes back to memory (accepted >= 0)
    int b, h;                 // sequence and value head of the item
    int tile_index;           // its state tile: (state slot) * H_v + h
    // trees of more than 64 nodes have no ancestor masks: the producer walks the accepted node's root path
    // through the parent array and leaves it here, root first
    uint8_t path[CP_WIDE_NODES];
};

struct CommitPipeSmem {
    CommitStage stage[CP_STAGES];
    int32_t par_scratch[CP_STAGES][CP_WIDE_NODES];
    uint8_t path_scratch[CP_STAGES][CP_WIDE_NODES];
    uint64_t full[CP_STAGES];
    uint64_t empty[CP_STAGES];
};

__global__ void __launch_bounds__(CP_THREADS, 1) commit_pipe_kernel(CommitArgs a, int n_items)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CommitPipeSmem &sm = *reinterpret_cast<CommitPipeSmem *>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < CP_STAGES; ++s) {
            ptx::mbar_init(&sm.full[s], 1);
            ptx::mbar_init(&sm.empty[s], 1);
        }
        ptx::fence_barrier_init();
    }
    grid_dependency_wait();  // the kernel before this one on the stream has finished: global memory may be read
    if (tid == 0) ptx::wait_deadline_init(a.wait_cycles);
    __syncthreads();
    grid_dependency_trigger();

    __nv_bfloat16 *S0 = static_cast<__nv_bfloat16 *>(a.S0);
    const uint32_t ub = a.u_half ? 2u : 4u;  // bytes of a U element
    const __nv_bfloat16 *kg = static_cast<const __nv_bfloat16 *>(a.k);
    const int group = a.H_v / a.H_qk;

    if (warp >= CP_CONSUMERS / 32) {
        // ------------------------------------------------------------------ producer warp
        const int s = warp - CP_CONSUMERS / 32;
        CommitStage &g = sm.stage[s];
        // (the parent array of the item being PREPARED lives outside the stage proper: the stage may still
        // be in the consumers' hands while the next item's path is walked)
        int32_t *g_par = sm.par_scratch[s];
        // The first item of a stage: its state tile depends on nothing but the item's number, so it is
        // put in flight before the chain accepted -> mask / log-gate -> path gates is walked (three or
        // four dependent loads, 4 us in a role trace, that would otherwise stand in front of the launch's
        // first bytes).
        const bool early = !a.snap_out && !a.state_index && (int)blockIdx.x + s * (int)gridDim.x < n_items;
        if (early && lane == 0) {
            ptx::mbar_expect_tx(&sm.full[s], CP_TILE_BYTES);
            ptx::bulk_g2s(g.tile, S0 + (size_t)(blockIdx.x + s * gridDim.x) * D * D, CP_TILE_BYTES, &sm.full[s]);
        }
        for (int kk = s;; kk += CP_STAGES) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const bool tile_issued = early && kk == s;
            int b, h;
            if (a.snap_out) {  // snapshot mode: item = (packed node, head); find the node's sequence
                const int t = item / a.H_v;
                h = item - t * a.H_v;
                int l = 0, r = a.B - 1;
                while (l < r) {
                    const int mid = (l + r + 1) >> 1;
                    if (a.node_offsets[mid] <= t) l = mid;
                    else r = mid - 1;
                }
                b = l;
            } else {
                b = item / a.H_v, h = item - b * a.H_v;
            }
            const int lo = a.node_offsets[b];
            const int n = a.node_offsets[b + 1] - lo;
            const int acc = a.snap_out ? item / a.H_v - lo : a.accepted[b];

            const int slot = state_slot(a.state_index, a.n_states, b);
            int bad = 0;
            if (slot < 0) {
                bad = TREEWY_SEQ_BAD_STATE;
            } else if (bad_offsets(lo, n, a.T)) {
                bad = TREEWY_SEQ_BAD_OFFSETS;
            } else if (n < 1 || n > a.max_nodes) {
                bad = TREEWY_SEQ_TOO_MANY_NODES;
            } else {
                int bp = 0;
                for (int i = lane; i < n; i += 32) {
                    const int p = a.parent[lo + i];
                    bp |= (p < -1 || p >= i);
                    if (!a.anc_mask) g_par[i] = p;
                }
                if (__any_sync(0xffffffffu, bp)) bad = TREEWY_SEQ_BAD_PARENT;
                else if (acc < -1 || acc >= n) bad = TREEWY_SEQ_BAD_ACCEPTED;
            }
            if (bad && h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);  // idempotent

            const bool work = !bad && (acc >= 0 || a.S_out_f32 != nullptr);
            unsigned long long mask = 0;
            float La = 0.f, wj = 0.f;
            int plen = work ? 0 : -1, cnt = 0, j = 0;
            uint8_t *g_path = sm.path_scratch[s];
            if (work && acc >= 0) {
                La = a.cum_log_gate[(size_t)(lo + acc) * a.H_v + h];
                if (a.anc_mask) {
                    mask = a.anc_mask[lo + acc];
                    plen = __popcll(mask);
                } else {  // walk up from the accepted node (parent[p] < p: ends), then lay the path out root first
                    __syncwarp();
                    if (lane == 0) {
                        int len = 0;
                        for (int p = acc; p >= 0; p = g_par[p]) ++len;
                        int e = len;
                        for (int p = acc; p >= 0; p = g_par[p]) g_path[--e] = (uint8_t)p;
                        plen = len;
                    }
                    __syncwarp();  // the path is written: every lane may read it
                    plen = __shfl_sync(0xffffffffu, plen, 0);
                }
                cnt = min(plen, CP_PCH);
                if (lane < cnt) {
                    j = a.anc_mask ? nth_set_bit(mask, lane) : (int)g_path[lane];
                    wj = expf(La - a.cum_log_gate[(size_t)(lo + j) * a.H_v + h]);
                }
            }
            // the stage must have been drained by the consumers' last store
            if (!ptx::mbar_wait(&sm.empty[s], ((kk / CP_STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], TREEWY_SEQ_TIMEOUT);
                break;
            }
            if (lane < cnt) g.w[lane] = wj;
            if (!a.anc_mask && plen > CP_PCH)  // (only a deep path's tail is read from the stage)
                for (int q = lane; q < plen; q += 32) g.path[q] = g_path[q];
            if (lane == 0) {
                g.mask = mask, g.La = La, g.ga = expf(La), g.plen = plen;
                g.store_tile = (acc >= 0);
                g.b = b, g.h = h, g.tile_index = (slot < 0 ? 0 : slot) * a.H_v + h;
            }
            __syncwarp();
            if (!work) {  // (a tile issued ahead still lands before the phase completes; nobody reads it)
                if (lane == 0) ptx::mbar_arrive(&sm.full[s]);
                continue;
            }
            if (lane == 0) {
                ptx::mbar_arrive_expect_tx(&sm.full[s], (tile_issued ? 0u : CP_TILE_BYTES) + cnt * (D * 2 + D * ub));
                if (!tile_issued)
                    ptx::bulk_g2s(g.tile, S0 + ((size_t)slot * a.H_v + h) * D * D, CP_TILE_BYTES, &sm.full[s]);
            }
            __syncwarp();
            if (lane < cnt) {
                ptx::bulk_g2s(g.krow[lane], kg + ((size_t)(lo + j) * a.H_qk + h / group) * D, D * 2,
                              &sm.full[s]);
                ptx::bulk_g2s(g.urow[lane], static_cast<const char *>(a.U) + ((size_t)(lo + j) * a.H_v + h) * D * ub, D * ub,
                              &sm.full[s]);
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int cc = tid & 15, r0 = tid >> 4;
    int pending = -1;  // stage whose bulk store may still be reading shared memory (tid 0)
    for (int kk = 0;; ++kk) {
        const int item = blockIdx.x + kk * gridDim.x;
        if (item >= n_items) break;
        const int s = kk % CP_STAGES;
        CommitStage &g = sm.stage[s];
        if (!ptx::mbar_wait(&sm.full[s], (kk / CP_STAGES) & 1)) {
            if (tid == 0 && a.seq_status && !a.snap_out) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
            break;
        }
        const int plen = g.plen;
        const int store_tile = g.store_tile;
        if (plen >= 0) {
            const int b = g.b, h = g.h;
            float acc[8][8];
            const float ga = g.ga;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const uint4 x = *reinterpret_cast<const uint4 *>(&g.tile[(r0 + 16 * it) * D + cc * 8]);
                widen8(x, acc[it]);
                if (store_tile) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[it][e] *= ga;
                }
            }
            const int cnt = min(plen, CP_PCH);
            for (int p = 0; p < cnt; ++p) {
                const float w = g.w[p];
                float kf[8];
                widen8(*reinterpret_cast<const uint4 *>(&g.krow[p][cc * 8]), kf);
#pragma unroll
                for (int e = 0; e < 8; ++e) kf[e] *= w;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const float u = a.u_half ? __half2float(reinterpret_cast<const __half *>(g.urow[p])[r0 + 16 * it])
                                             : g.urow[p][r0 + 16 * it];
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[it][e] = fmaf(u, kf[e], acc[it][e]);
                }
            }
            if (plen > CP_PCH) {  // deep path: remaining nodes straight from global memory
                const int lo = a.node_offsets[b];
                unsigned long long m = g.mask;
                for (int q = 0; q < CP_PCH; ++q) m &= m - 1;
                for (int q = CP_PCH; q < plen; ++q) {
                    const int j = a.anc_mask ? __ffsll((long long)m) - 1 : (int)g.path[q];
                    m &= m - 1;
                    const float w = expf(g.La - a.cum_log_gate[(size_t)(lo + j) * a.H_v + h]);
                    float kf[8];
                    widen8(*reinterpret_cast<const uint4 *>(
                               kg + ((size_t)(lo + j) * a.H_qk + h / group) * D + cc * 8),
                           kf);
#pragma unroll
                    for (int e = 0; e < 8; ++e) kf[e] *= w;
                    const size_t ur = ((size_t)(lo + j) * a.H_v + h) * D;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const float u = load_u(a.U, ur + r0 + 16 * it, a.u_half);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[it][e] = fmaf(u, kf[e], acc[it][e]);
                    }
                }
            }
            if (store_tile) {
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    uint4 y;
                    y.x = pack_bf16(acc[it][0], acc[it][1]), y.y = pack_bf16(acc[it][2], acc[it][3]);
                    y.z = pack_bf16(acc[it][4], acc[it][5]), y.w = pack_bf16(acc[it][6], acc[it][7]);
                    *reinterpret_cast<uint4 *>(&g.tile[(r0 + 16 * it) * D + cc * 8]) = y;
                }
                ptx::fence_proxy_async();
            }
            if (a.S_out_f32) {
                float *o = a.S_out_f32 + (size_t)item * D * D;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    float4 *dst = reinterpret_cast<float4 *>(o + (size_t)(r0 + 16 * it) * D + cc * 8);
                    dst[0] = make_float4(acc[it][0], acc[it][1], acc[it][2], acc[it][3]);
                    dst[1] = make_float4(acc[it][4], acc[it][5], acc[it][6], acc[it][7]);
                }
            }
        }
        ptx::named_sync(1, CP_CONSUMERS);  // every consumer is done with this stage
        if (tid == 0) {
            if (plen >= 0 && store_tile) {
                __nv_bfloat16 *dst = a.snap_out ? static_cast<__nv_bfloat16 *>(a.snap_out) + (size_t)item * D * D
                                                : S0 + (size_t)g.tile_index * D * D;
                ptx::bulk_s2g(dst, g.tile, CP_TILE_BYTES);
                ptx::bulk_commit_group();
                if (pending >= 0) {
                    ptx::bulk_wait_group_read<1>();  // the previous store has left its stage
                    ptx::mbar_arrive(&sm.empty[pending]);
                }
                pending = s;
            } else {
                if (pending >= 0) {
                    ptx::bulk_wait_group_read<0>();
                    ptx::mbar_arrive(&sm.empty[pending]);
                    pending = -1;
                }
                ptx::mbar_arrive(&sm.empty[s]);
            }
        }
    }
    if (tid == 0) ptx::bulk_wait_group<0>();
}

cudaError_t launch_commit_pipe(const CommitArgs &a, cudaStream_t stream)
{
    const long long n_items = (long long)(a.snap_out ? a.T : a.B) * a.H_v;
    if (n_items == 0) return cudaSuccess;
    int dev = 0, sms = 0;
    cudaError_t e = current_device_sms(&dev, &sms);
    if (e != cudaSuccess) return e;
    static_assert(sizeof(CommitPipeSmem) <= 227 * 1024, "shared memory of one CTA");
    const int smem = (int)sizeof(CommitPipeSmem);
    e = ensure_dynamic_smem(reinterpret_cast<const void *>(commit_pipe_kernel), smem, dev);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    return launch_dependent(commit_pipe_kernel, dim3(grid), dim3(CP_THREADS), smem, stream, a, (int)n_items);
}

}  // namespace treewy
