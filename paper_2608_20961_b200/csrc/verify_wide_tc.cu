// treewy_verify_wide, bf16 kernel for draft trees of up to 128 nodes (Section 3: Eq. 2 and the
// read-out hold for any N; the draft window is a serving parameter, Section 4), with the dense
// contractions on the tcgen05 tensor cores:
//
//   D1  = S0 [Q;K]^T     M = 128 state rows, N = 256 (128 q rows, 128 k rows), K = 128   -> S0 q_i, S0 k_i
//   Gqk = Q K^T, Gkk = K K^T     M = 128 nodes, N = 128 nodes, K = 128                   -> q_i.k_j, k_i.k_j
//
// all three accumulated in tensor memory (256 + 128 + 128 = 512 columns: one item at a time).  A node
// of such a tree has no 64-bit ancestor mask; the producer warp walks the parent array once per item
// and hands over four-word masks, depths and the level order.  The triangular system itself is solved
// on the CUDA cores:
//
//   lists     the thread whose tensor-memory lane holds row i of a Gram block picks node i's ancestors
//             out of it (through a private line of shared memory, so that they can be taken by index):
//             A[i][d] = beta_i e^{L_i - L_j} k_i.k_j, P[i][d] = e^{L_i - L_j} q_i.k_j, j the ancestor of
//             depth d (ancestors in index order are in depth order);
//   r, o0     thread c = tensor-memory lane c = element c of d_v:  r_i[c] = beta_i v_i[c] - beta_i g_i (S0 k_i)[c]
//             and o0_i[c] = g_i (S0 q_i)[c] into two [node][c] tiles of shared memory; tensor memory is
//             not needed after this;
//   solve     level by level (nodes of one depth do not depend on each other): ONE WARP PER NODE, a lane
//             holding four elements of d_v, so that the coefficients and indices, which are the same for
//             all 128 elements, are fetched once per node and not once per 32 elements:
//             u_i = r_i - sum_d A[i][d] u_{j_d},  o_i = o0_i + sum_d P[i][d] u_{j_d} + (q_i.k_i) u_i;
//             u_i replaces r_i in its tile, both rows leave for global memory as 512 / 256 contiguous bytes.
//             (A first version gave every node to four warps of 32 elements each: 37 k warp instructions
//             and 20 k cycles per item in this phase alone.)
//
// The lists keep WT_DCAP entries per node, which covers the trees speculative decoding drafts (wide,
// a handful of levels).  A tree with a deeper path takes a slower route through the same kernel: no
// lists, every coefficient read from tensor memory when it is needed.
//
// Shared memory holds one item.  The q / k tiles are free again as soon as the tensor core has read them,
// so the next item's q / k rows land during this item's solve; the o0 tile lies over the S0 and v
// tiles, whose refill waits for the end of the solve (the next MMAs then wait for S0 only).  Every mbarrier
// wait is bounded by the kernel's deadline (TREEWY_SEQ_TIMEOUT on give-up).
#include <cuda.h>

#include <cstddef>
#include <type_traits>

#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

namespace {

constexpr int WN = TREEWY_MAX_NODES_WIDE;
constexpr int WT_DCAP = WIDE_TC_MAX_DEPTH;
constexpr int WT_GROUPS = 4;               // consumer groups of 128 threads (thread = element c of d_v)
constexpr int WT_CONS = WT_GROUPS * 128;
constexpr int WT_CWARPS = WT_CONS / 32;
constexpr int WT_PROD_WARP = WT_CWARPS, WT_MMA_WARP = WT_CWARPS + 1;
constexpr int WT_THREADS = WT_CONS + 64;
constexpr uint32_t WT_TMEM_COLS = 512;
constexpr int TM_SQ = 0, TM_SK = WN, TM_GQK = 2 * WN, TM_GKK = 3 * WN;

// what the producer warp says about an item (two of them: the next item's is written while this one's is read)
struct WtMeta {
    alignas(16) uint32_t mask[WN][4];       // ancestor-or-self (read and written 16 bytes at a time)
    float L[WN], beta[WN], bg[WN], g[WN];   // log-gate, beta, beta g, g per node
    int n, lo, h, b, maxd;      // n = 0: nothing to verify here (malformed sequence)
    int deep;                   // some path has more than WT_DCAP ancestors: no lists, coefficients on demand
    int lvl[WN + 2];            // first position of every level in `order`; lvl[maxd + 1] = n
    uint8_t order[WN];          // nodes sorted by (depth, index)
};
static_assert(offsetof(WtMeta, mask) % 16 == 0, "mask rows are accessed as uint4");

constexpr int QK_HALF = 2 * WN * 128;                 // q rows then k rows of one 64-column half
constexpr int OFF_QK = 0, OFF_S0 = 2 * QK_HALF, S0_HALF = D * 128;
constexpr int OFF_V = OFF_S0 + 2 * S0_HALF;           // v rows [128][128] bf16
constexpr int OFF_U = OFF_V + WN * D * 2;             // r_i, then u_i: [node][c] fp32
constexpr int OFF_AP = OFF_U + WN * D * 4;            // (A, P)[node][d]
constexpr int OFF_IDX = OFF_AP + WN * WT_DCAP * 8;    // ancestor index [node][d]
constexpr int OFF_PSELF = OFF_IDX + WN * WT_DCAP;     // q_i . k_i
constexpr int OFF_PAR = OFF_PSELF + WN * 4;           // producer scratch: the sequence's parent array
constexpr int OFF_O0 = OFF_S0;                        // o0_i = g_i S0 q_i: [node][c] fp32 over the S0 and v tiles
static_assert(OFF_V == OFF_S0 + 2 * S0_HALF && 2 * S0_HALF + WN * D * 2 >= WN * D * 4, "the o0 tile fits over S0 | v");
constexpr int META_BYTES = ((int)sizeof(WtMeta) + 15) / 16 * 16;
constexpr int OFF_META = OFF_PAR + WN * 4;
static_assert(OFF_META % 16 == 0 && META_BYTES % 16 == 0 && OFF_AP % 8 == 0, "alignment of vector accesses");
constexpr int OFF_BAR = OFF_META + 2 * META_BYTES;
constexpr int N_BARS = 12;
constexpr int SMEM_BYTES = OFF_BAR + N_BARS * 8 + 16 + 1024;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
constexpr uint32_t TX_QK = 2 * QK_HALF, TX_S0 = 2 * S0_HALF, TX_V = WN * D * 2;

__device__ __forceinline__ void store_o4(float *p, const float4 &o) { *reinterpret_cast<float4 *>(p) = o; }
__device__ __forceinline__ void store_o4(__nv_bfloat16 *p, const float4 &o)
{
    *reinterpret_cast<uint2 *>(p) = make_uint2(pack_bf16(o.x, o.y), pack_bf16(o.z, o.w));
}

template <typename TOut>
__global__ void __launch_bounds__(WT_THREADS, 1)
verify_wide_tc_kernel(VerifyArgs a, int n_items, const __grid_constant__ CUtensorMap tmS0,
                      const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV)
{
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + OFF_BAR);
    uint64_t *full_qk = bars, *free_qk = bars + 1, *full_v = bars + 2, *free_sv = bars + 3;
    uint64_t *mma_done = bars + 4, *tmem_free = bars + 5, *meta_full = bars + 6, *meta_free = bars + 8;
    uint64_t *full_s0 = bars + 10;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + N_BARS);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        ptx::mbar_init(full_qk, 1), ptx::mbar_init(free_qk, 1);
        ptx::mbar_init(full_s0, 1), ptx::mbar_init(full_v, 1), ptx::mbar_init(free_sv, WT_CWARPS);
        ptx::mbar_init(mma_done, 1), ptx::mbar_init(tmem_free, WT_CWARPS);
        for (int x = 0; x < 2; ++x) {
            ptx::mbar_init(&meta_full[x], 1);
            ptx::mbar_init(&meta_free[x], WT_CWARPS + 1);  // the consumer warps and the MMA warp
        }
        ptx::fence_barrier_init();
    }
    if (tid == 32) {
        ptx::prefetch_tmap(&tmS0), ptx::prefetch_tmap(&tmQ);
        ptx::prefetch_tmap(&tmK), ptx::prefetch_tmap(&tmV);
    }
    if (warp == WT_MMA_WARP) {
        ptx::tmem_alloc(tmem_slot, WT_TMEM_COLS);
        ptx::tmem_relinquish();
        ptx::tc_fence_before_sync();
    }
    grid_dependency_wait();  // the kernel before this one on the stream has finished: global memory may be read
    if (tid == 0) ptx::wait_deadline_init(a.wait_cycles);
    __syncthreads();
    grid_dependency_trigger();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    auto meta_of = [&](int kk) { return reinterpret_cast<WtMeta *>(smem + OFF_META + (kk & 1) * META_BYTES); };

    if (warp == WT_PROD_WARP) {
        // ------------------------------------------------------------------ producer warp
        int32_t *spar = reinterpret_cast<int32_t *>(smem + OFF_PAR);
        const int group = a.H_v / a.H_qk;
        uint32_t np = 0;  // items loaded so far: phase of the load barriers
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = (int)blockIdx.x + kk * (int)gridDim.x;
            if (item >= n_items) break;
            const int b = item / a.H_v, h = item - b * a.H_v;
            const int lo = a.node_offsets[b];
            const int n = a.node_offsets[b + 1] - lo;
            int bad = bad_offsets(lo, n, a.T) ? TREEWY_SEQ_BAD_OFFSETS
                      : (n < 1 || n > a.max_nodes) ? TREEWY_SEQ_TOO_MANY_NODES : 0;
            int par[4];
            if (!bad) {
                bool bp = false;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = lane + 32 * r;
                    par[r] = i < n ? a.parent[lo + i] : -1;
                    bp |= i < n && (par[r] < -1 || par[r] >= i);
                }
                if (__any_sync(0xffffffffu, bp)) bad = TREEWY_SEQ_BAD_PARENT;
            }
            if (bad && h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
            // the meta block of two items ago must have been read by everybody
            if (!ptx::mbar_wait(&meta_free[kk & 1], ((kk >> 1) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], TREEWY_SEQ_TIMEOUT);
                break;
            }
            WtMeta *m = meta_of(kk);
            int maxd = 0;
            bool run = !bad;
            if (run) {
#pragma unroll
                for (int r = 0; r < 4; ++r) spar[lane + 32 * r] = par[r];
                __syncwarp();
                int dep[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {  // node i walks up its root path: mask and depth
                    const int i = lane + 32 * r;
                    unsigned long long mlo = 0ull, mhi = 0ull;
                    int d = 0;
                    if (i < n) {
                        if (i < 64) mlo = 1ull << i;
                        else mhi = 1ull << (i - 64);
                        for (int p = par[r]; p >= 0; p = spar[p]) {  // parent[p] < p: ends
                            if (p < 64) mlo |= 1ull << p;
                            else mhi |= 1ull << (p - 64);
                            ++d;
                        }
                        *reinterpret_cast<uint4 *>(m->mask[i]) =
                            make_uint4((uint32_t)mlo, (uint32_t)(mlo >> 32), (uint32_t)mhi, (uint32_t)(mhi >> 32));
                    }
                    dep[r] = i < n ? d : -1;
                    maxd = max(maxd, d);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) maxd = max(maxd, __shfl_xor_sync(0xffffffffu, maxd, o));
                {
                    int pos = 0;
#pragma unroll 1
                    for (int dd = 0; dd <= maxd; ++dd) {  // counting sort by depth; index order inside a level
                        if (lane == 0) m->lvl[dd] = pos;
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const uint32_t bal = __ballot_sync(0xffffffffu, dep[r] == dd);
                            if (dep[r] == dd) m->order[pos + __popc(bal & ((1u << lane) - 1u))] = (uint8_t)(lane + 32 * r);
                            pos += __popc(bal);
                        }
                    }
                    if (lane == 0) m->lvl[maxd + 1] = pos;
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const int i = lane + 32 * r;
                        if (i < n) {
                            const float Lv = a.cum_log_gate[(size_t)(lo + i) * a.H_v + h];
                            const float bv = a.beta[(size_t)(lo + i) * a.H_v + h];
                            const float gv = expf(Lv);
                            m->L[i] = Lv, m->beta[i] = bv, m->g[i] = gv, m->bg[i] = bv * gv;
                        }
                    }
                }
            }
            if (lane == 0) m->n = run ? n : 0, m->lo = lo, m->h = h, m->b = b, m->maxd = maxd, m->deep = maxd > WT_DCAP;
            __syncwarp();
            if (run) {
                const int hq = h / group;
                // The q / k tiles are free once the tensor core has read them, early in the previous item: its
                // solve hides their refill.  The S0 and v tiles carry that item's o0 tile until its solve has
                // ended; S0 is what the next MMAs then wait for, v lands behind them.
                if (!ptx::mbar_wait(free_qk, (np & 1) ^ 1)) break;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(full_qk, TX_QK);
                    ptx::tma_load_2d(smem + OFF_QK, &tmQ, hq * D, lo, full_qk);
                    ptx::tma_load_2d(smem + OFF_QK + QK_HALF, &tmQ, hq * D + 64, lo, full_qk);
                    ptx::tma_load_2d(smem + OFF_QK + WN * 128, &tmK, hq * D, lo, full_qk);
                    ptx::tma_load_2d(smem + OFF_QK + QK_HALF + WN * 128, &tmK, hq * D + 64, lo, full_qk);
                }
                if (!ptx::mbar_wait(free_sv, (np & 1) ^ 1)) break;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(full_s0, TX_S0);
                    ptx::tma_load_2d(smem + OFF_S0, &tmS0, 0, item * D, full_s0);
                    ptx::tma_load_2d(smem + OFF_S0 + S0_HALF, &tmS0, 64, item * D, full_s0);
                    ptx::mbar_arrive_expect_tx(full_v, TX_V);
                    ptx::tma_load_2d(smem + OFF_V, &tmV, h * D, lo, full_v);
                }
                ++np;
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&meta_full[kk & 1]);
        }
    } else if (warp == WT_MMA_WARP) {
        // ------------------------------------------------------------------ MMA warp
        constexpr uint32_t idesc1 = ptx::umma_idesc_bf16_f32(128, 2 * WN);
        constexpr uint32_t idesc2 = ptx::umma_idesc_bf16_f32(128, WN);
        uint32_t np = 0;
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = (int)blockIdx.x + kk * (int)gridDim.x;
            if (item >= n_items) break;
            if (!ptx::mbar_wait(&meta_full[kk & 1], (kk >> 1) & 1)) break;
            const int n = meta_of(kk)->n;
            if (n > 0) {
                if (!ptx::mbar_wait(full_s0, np & 1)) break;
                if (!ptx::mbar_wait(full_qk, np & 1)) break;
                if (!ptx::mbar_wait(tmem_free, (np & 1) ^ 1)) break;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t qk = ptx::smem_u32(smem + OFF_QK), s0 = ptx::smem_u32(smem + OFF_S0);
#pragma unroll 1
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t ko = (ks >> 2) * QK_HALF + (ks & 3) * 32;
                        const uint64_t dq = ptx::umma_desc_k_sw128(qk + ko);               // q rows (then k rows)
                        const uint64_t dk = ptx::umma_desc_k_sw128(qk + ko + WN * 128);    // k rows
                        const uint64_t ds = ptx::umma_desc_k_sw128(s0 + (ks >> 2) * S0_HALF + (ks & 3) * 32);
                        ptx::umma_bf16(tmem_base + TM_SQ, ds, dq, idesc1, ks > 0);
                        ptx::umma_bf16(tmem_base + TM_GQK, dq, dk, idesc2, ks > 0);
                        ptx::umma_bf16(tmem_base + TM_GKK, dk, dk, idesc2, ks > 0);
                    }
                    ptx::umma_commit(free_qk);  // the tiles have been read
                    ptx::umma_commit(mma_done);
                }
                __syncwarp();
                ++np;
            }
            if (lane == 0) ptx::mbar_arrive(&meta_free[kk & 1]);
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int q4 = warp & 3, grp = warp >> 2;
        const int c = q4 * 32 + lane;  // element of d_v = TMEM lane (state products); node = TMEM lane (Gram blocks)
        const uint32_t tl = tmem_base + ((uint32_t)(q4 * 32) << 16);
        float *Ut = reinterpret_cast<float *>(smem + OFF_U);
        float2 *AP = reinterpret_cast<float2 *>(smem + OFF_AP);
        unsigned char *IDX = smem + OFF_IDX;
        float *pself = reinterpret_cast<float *>(smem + OFF_PSELF);
        float *O0 = reinterpret_cast<float *>(smem + OFF_O0);
        const __nv_bfloat16 *Vt = reinterpret_cast<const __nv_bfloat16 *>(smem + OFF_V);
        TOut *Og = static_cast<TOut *>(a.O);
        float *Ug = static_cast<float *>(a.U);
        const size_t rs = (size_t)a.H_v * D;
        uint32_t np = 0;
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = (int)blockIdx.x + kk * (int)gridDim.x;
            if (item >= n_items) break;
            if (!ptx::mbar_wait(&meta_full[kk & 1], (kk >> 1) & 1)) {
                if (tid == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            const WtMeta *m = meta_of(kk);
            const int n = m->n;
            if (n == 0) {
                ptx::mbar_arrive_warp(&meta_free[kk & 1]);
                continue;
            }
            if (!ptx::mbar_wait(mma_done, np & 1)) {
                if (tid == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            ptx::tc_fence_after_sync();
            const bool deep = m->deep != 0;
            if (!deep) {
                // ---- lists: this thread's Gram row (node c), half of its columns; even groups take
                // q_c . k_j (P), odd groups k_c . k_j (A)
                const int i = c, mat = grp & 1, ch = grp >> 1;
                const uint4 mw = *reinterpret_cast<const uint4 *>(m->mask[i < n ? i : 0]);
                const uint32_t self = 1u << (i & 31), sw = i >> 5;  // proper ancestors: the self bit goes
                const uint32_t p0 = mw.x & ~(sw == 0 ? self : 0u), p1 = mw.y & ~(sw == 1 ? self : 0u);
                const uint32_t p2 = mw.z & ~(sw == 2 ? self : 0u), p3 = mw.w & ~(sw == 3 ? self : 0u);
                const uint32_t words[2] = {ch ? p2 : p0, ch ? p3 : p1};  // this thread's 64 columns
                const float Li = m->L[i < n ? i : 0], scale = mat ? m->beta[i < n ? i : 0] : 1.f;
                int pos = ch ? __popc(p0) + __popc(p1) : 0;
                // The 32 entries of a chunk go from tensor memory to a private 128-byte line of shared memory
                // (the tile that later holds r and u is idle now), 16-byte pieces rotated by the lane so that
                // the stores of a quarter warp fall on different banks; the few ancestors among them are then
                // picked by index.  (Testing all 32 columns in registers instead cost 900 instructions per thread.)
                float *line = Ut + tid * 32;
#pragma unroll
                for (int cq = 0; cq < 2; ++cq) {
                    const int c0 = 64 * ch + 32 * cq;
                    if (c0 < n) {  // (columns at or beyond n hold other sequences' rows: never an ancestor)
                        uint32_t g[32];
                        ptx::tmem_ld32(tl + (mat ? TM_GKK : TM_GQK) + c0, g);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            *reinterpret_cast<uint4 *>(line + 4 * (q ^ (lane & 7))) =
                                make_uint4(g[4 * q], g[4 * q + 1], g[4 * q + 2], g[4 * q + 3]);
                        auto entry = [&](int cc) { return line[4 * ((cc >> 2) ^ (lane & 7)) + (cc & 3)]; };
                        if (i < n) {
                            uint32_t word = words[cq];
#pragma unroll 1
                            while (word) {
                                const int cc = __ffs((int)word) - 1;
                                word &= word - 1;
                                const float val = scale * __expf(Li - m->L[c0 + cc]) * entry(cc);
                                if (mat) {
                                    AP[i * WT_DCAP + pos].x = val;
                                } else {
                                    AP[i * WT_DCAP + pos].y = val;
                                    IDX[i * WT_DCAP + pos] = (unsigned char)(c0 + cc);
                                }
                                ++pos;
                            }
                            if (!mat && (i >> 5) == (c0 >> 5)) pself[i] = entry(i & 31);  // q_i . k_i
                        }
                    }
                }
            }
            {
                // ---- r_i[c] and o0_i[c] for the nodes 32 grp .. 32 grp + 31 of this thread's group.  The o0
                // tile lies over the S0 and v tiles: every v element is in a register before the first o0
                // row is written (the same barrier says that the lines of the list phase have been read).
                if (!ptx::mbar_wait(full_v, np & 1)) {
                    if (tid == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                    break;
                }
                const int i0 = 32 * grp;
                float vv[32];
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) vv[jj] = i0 + jj < n ? __bfloat162float(Vt[(i0 + jj) * D + c]) : 0.f;
                ptx::named_sync(1, WT_CONS);
                if (i0 < n) {
                    uint32_t sx[32];
                    ptx::tmem_ld32(tl + TM_SK + i0, sx);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int i = i0 + jj;
                        if (i < n) Ut[i * D + c] = fmaf(-m->bg[i], __uint_as_float(sx[jj]), m->beta[i] * vv[jj]);
                    }
                    ptx::tmem_ld32(tl + TM_SQ + i0, sx);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int i = i0 + jj;
                        if (i < n) O0[i * D + c] = m->g[i] * __uint_as_float(sx[jj]);
                    }
                }
                if (!deep) {
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive_warp(tmem_free);  // tensor memory has been read out
                }
            }
            ptx::named_sync(1, WT_CONS);  // lists, q_i . k_i, r and o0 are in place
            // ---- the solve, level by level, a warp per node, a lane per four elements of d_v
            const int lo = m->lo, h = m->h, maxd = m->maxd;
            const size_t row0 = ((size_t)lo * a.H_v + h) * D + 4 * lane;
            if (deep) {
                // A tree with a path of more than WT_DCAP ancestors (a chain, a comb: not what drafting
                // produces, but a legal input): no lists.  The Gram blocks are still in tensor memory, where
                // row i is held by lane i % 32 of the warps of quarter i / 32; so a node goes to a warp of its
                // own quarter, which reads one column at a time and passes the entry round by shuffle.  Slow
                // (two tensor-memory reads per ancestor), correct for any tree.
#pragma unroll 1
                for (int lv = 0; lv <= maxd; ++lv) {
                    const int p1 = m->lvl[lv + 1];
                    int mine = 0;
#pragma unroll 1
                    for (int p = m->lvl[lv]; p < p1; ++p) {
                        const int i = m->order[p];
                        if ((i >> 5) != q4) continue;
                        if ((mine++ & (WT_GROUPS - 1)) != grp) continue;
                        const uint4 mw = *reinterpret_cast<const uint4 *>(m->mask[i]);
                        uint32_t pw[4] = {mw.x, mw.y, mw.z, mw.w};
                        const float Li = m->L[i], bi = m->beta[i];
                        float4 u = reinterpret_cast<const float4 *>(Ut + i * D)[lane];
                        float4 o = reinterpret_cast<const float4 *>(O0 + i * D)[lane];
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            uint32_t word = pw[w];
                            if (w == (i >> 5)) word &= ~(1u << (i & 31));  // proper ancestors
#pragma unroll 1
                            while (word) {
                                const int j = 32 * w + __ffs((int)word) - 1;
                                word &= word - 1;
                                const uint32_t kkv = ptx::tmem_ld1(tl + TM_GKK + j), qkv = ptx::tmem_ld1(tl + TM_GQK + j);
                                ptx::tmem_wait_ld();
                                const float kk = __uint_as_float(__shfl_sync(0xffffffffu, kkv, i & 31));
                                const float qk = __uint_as_float(__shfl_sync(0xffffffffu, qkv, i & 31));
                                const float e = __expf(Li - m->L[j]), ca = bi * e * kk, cp = e * qk;
                                const float4 uj = reinterpret_cast<const float4 *>(Ut + j * D)[lane];
                                u.x = fmaf(-ca, uj.x, u.x), u.y = fmaf(-ca, uj.y, u.y);
                                u.z = fmaf(-ca, uj.z, u.z), u.w = fmaf(-ca, uj.w, u.w);
                                o.x = fmaf(cp, uj.x, o.x), o.y = fmaf(cp, uj.y, o.y);
                                o.z = fmaf(cp, uj.z, o.z), o.w = fmaf(cp, uj.w, o.w);
                            }
                        }
                        const uint32_t psv = ptx::tmem_ld1(tl + TM_GQK + i);
                        ptx::tmem_wait_ld();
                        const float ps = __uint_as_float(__shfl_sync(0xffffffffu, psv, i & 31));  // q_i . k_i
                        o.x = fmaf(ps, u.x, o.x), o.y = fmaf(ps, u.y, o.y), o.z = fmaf(ps, u.z, o.z), o.w = fmaf(ps, u.w, o.w);
                        reinterpret_cast<float4 *>(Ut + i * D)[lane] = u;
                        *reinterpret_cast<float4 *>(Ug + row0 + (size_t)i * rs) = u;
                        store_o4(Og + row0 + (size_t)i * rs, o);
                    }
                    ptx::named_sync(1, WT_CONS);  // the level's u rows are visible to every warp
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(tmem_free);  // the Gram blocks were read to the end
            }
#pragma unroll 1
            for (int lv = 0; lv <= (deep ? -1 : maxd); ++lv) {
                const int p1 = m->lvl[lv + 1];
                // (a node is a chain of dependent shared-memory reads -- order -> lists -> u_j -- so a warp
                // takes two nodes of the level side by side where the level has them)
                auto nodes = [&](auto nb_tag, int p) {
                    constexpr int NB = decltype(nb_tag)::value;
                    int ii[NB];
                    float4 u[NB], o[NB];
#pragma unroll
                    for (int t = 0; t < NB; ++t) ii[t] = m->order[p + t * WT_CWARPS];
#pragma unroll
                    for (int t = 0; t < NB; ++t) {
                        u[t] = reinterpret_cast<const float4 *>(Ut + ii[t] * D)[lane];
                        o[t] = reinterpret_cast<const float4 *>(O0 + ii[t] * D)[lane];
                    }
#pragma unroll 2
                    for (int d = 0; d < lv; ++d) {
#pragma unroll
                        for (int t = 0; t < NB; ++t) {
                            const float2 co = AP[ii[t] * WT_DCAP + d];
                            const float4 uj = reinterpret_cast<const float4 *>(Ut + (int)IDX[ii[t] * WT_DCAP + d] * D)[lane];
                            u[t].x = fmaf(-co.x, uj.x, u[t].x), u[t].y = fmaf(-co.x, uj.y, u[t].y);
                            u[t].z = fmaf(-co.x, uj.z, u[t].z), u[t].w = fmaf(-co.x, uj.w, u[t].w);
                            o[t].x = fmaf(co.y, uj.x, o[t].x), o[t].y = fmaf(co.y, uj.y, o[t].y);
                            o[t].z = fmaf(co.y, uj.z, o[t].z), o[t].w = fmaf(co.y, uj.w, o[t].w);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < NB; ++t) {
                        const float ps = pself[ii[t]];
                        o[t].x = fmaf(ps, u[t].x, o[t].x), o[t].y = fmaf(ps, u[t].y, o[t].y);
                        o[t].z = fmaf(ps, u[t].z, o[t].z), o[t].w = fmaf(ps, u[t].w, o[t].w);
                        reinterpret_cast<float4 *>(Ut + ii[t] * D)[lane] = u[t];
                        *reinterpret_cast<float4 *>(Ug + row0 + (size_t)ii[t] * rs) = u[t];
                        store_o4(Og + row0 + (size_t)ii[t] * rs, o[t]);
                    }
                };
                int p = m->lvl[lv] + warp;
#pragma unroll 1
                for (; p + WT_CWARPS < p1; p += 2 * WT_CWARPS) nodes(std::integral_constant<int, 2>{}, p);
                if (p < p1) nodes(std::integral_constant<int, 1>{}, p);
                ptx::named_sync(1, WT_CONS);  // the level's u rows are visible to every warp
            }
            ptx::mbar_arrive_warp(free_sv);  // the o0 tile has been read: the next item's S0 tile and v rows may land
            ptx::mbar_arrive_warp(&meta_free[kk & 1]);
            ++np;
        }
    }

    // common exit: tensor memory goes back once every role is done with it
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == WT_MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, WT_TMEM_COLS);
    }
}

template <typename TOut> cudaError_t launch_wt(const VerifyArgs &a, cudaStream_t stream)
{
    const long long n_items = (long long)a.B * a.H_v;
    VerifyMaps m;
    if (!make_verify_maps(&m, a.S0, a.q, a.k, a.v, n_items, a.T, a.H_v, a.H_qk, WN)) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = current_device_sms(&dev, &sms);
    if (e != cudaSuccess) return e;
    e = ensure_dynamic_smem(reinterpret_cast<const void *>(verify_wide_tc_kernel<TOut>), SMEM_BYTES, dev);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    return launch_dependent(verify_wide_tc_kernel<TOut>, dim3(grid), dim3(WT_THREADS), SMEM_BYTES, stream, a,
                            (int)n_items, m.S0, m.Q, m.K, m.V);
}

}  // namespace

cudaError_t launch_verify_wide_tc(const VerifyArgs &a, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0 || a.T == 0) return cudaSuccess;
    return od == TREEWY_F32 ? launch_wt<float>(a, stream) : launch_wt<__nv_bfloat16>(a, stream);
}

}  // namespace treewy
