// treewy_verify, bf16 production kernel for trees of 33..64 nodes (Section 3: Eq. 2 and the
// read-out).  Same method as the up-to-32-node kernel -- both contractions on tcgen05, the
// triangular solve replaced by per-node path inverses T = (I + A)^-1, W = P T -- laid out for
// twice the nodes, where shared memory is the scarce resource:
//
//   * R^T (the A operand of the stage-2 products) never touches shared memory: thread c writes
//     its row (hi and lo tf32 parts) into TENSOR memory with tcgen05.st, over the Gram columns
//     it has already consumed, and the stage-2 MMAs take A from tensor memory;
//   * the T / W operand tiles (4 x 16 KiB, fp32 rows of 64 columns as two 128-byte-swizzled
//     atoms) overlay the dead [Q;K] and S0 tiles exactly; each row is zeroed and filled by the
//     one thread that computes it, so no fill barrier is needed;
//   * the read-out needs no separate pass: g_i (S0 q_i) is scaled in place in tensor memory and
//     the R^T W^T product accumulates on top of it, U lands over the consumed S0 k columns.
//
// One consumer group of 128 threads (thread c = TMEM lane c = row c of d_v), software-pipelined:
// the front half of item k+1 (lists, T / W rows, R^T) runs before the epilogue of item k, so the
// stage-2 MMAs are never waited for.  Two load stages, two TMEM buffers of 256 columns.
#include <cuda.h>

#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

namespace {

constexpr int V6_NP = 64;
constexpr int V6_GROUP = 128;
constexpr int V6_STAGES = 2;
constexpr int V6_TBUF = 2;
constexpr int V6_MMA1_WARP = V6_GROUP / 32, V6_MMA2_WARP = V6_MMA1_WARP + 1, V6_PROD_WARP0 = V6_MMA2_WARP + 1;
constexpr int V6_THREADS = V6_GROUP + 64 + 32 * V6_STAGES;
// stage: [Q;K] tile (128 rows) | S0 tile | v rows | meta
constexpr int V6_QK_HALF = 2 * V6_NP * 128, V6_QK_BYTES = 2 * V6_QK_HALF;
constexpr int V6_S0_HALF = D * 128, V6_S0_BYTES = 2 * V6_S0_HALF;
constexpr int V6_V_BYTES = V6_NP * D * 2;
constexpr int V6_OFF_S0 = V6_QK_BYTES, V6_OFF_V = V6_OFF_S0 + V6_S0_BYTES, V6_OFF_META = V6_OFF_V + V6_V_BYTES;
constexpr int V6_META_BYTES = V6_NP * 16 + 16;
constexpr int V6_STAGE_BYTES = (V6_OFF_META + V6_META_BYTES + 1023) / 1024 * 1024;
constexpr uint32_t V6_TX_BYTES = V6_QK_BYTES + V6_S0_BYTES + V6_V_BYTES;
// overlays on the dead tiles: raw Gram rows first, then the four operand tiles
constexpr int V6_RLD = V6_NP + 4;
// The stage-2 B operand is [W;T]: 128 rows (W rows above T rows) of 64 fp32 columns, as two
// 128-byte-swizzled atoms of 128 rows each, once for the hi parts and once for the lo parts; one
// MMA then yields O and U together.
constexpr int V6_TILE = V6_NP * 256;       // bytes of one 64-row operand [64 rows][64 cols]
constexpr int V6_ATOM = 2 * V6_NP * 128;   // one atom of the stacked operand: 128 rows x 128 bytes
constexpr int V6_OFF_X_HI = 0, V6_OFF_X_LO = 2 * V6_ATOM;
constexpr int V6_OFF_W_HI = V6_OFF_X_HI, V6_OFF_T_HI = V6_OFF_X_HI + V6_NP * 128;
constexpr int V6_OFF_W_LO = V6_OFF_X_LO, V6_OFF_T_LO = V6_OFF_X_LO + V6_NP * 128;
static_assert(4 * V6_TILE <= V6_QK_BYTES + V6_S0_BYTES, "operand tiles fit the dead tiles");
static_assert(2 * V6_NP * V6_RLD * 4 <= V6_QK_BYTES + V6_S0_BYTES, "raw Gram rows fit the dead tiles");
// group-private: path lists [d / 4][node][d % 4], per-node scalars, ancestor indices
constexpr int V6_GP_AP = 0, V6_GP_PP = V6_NP * V6_NP * 4, V6_GP_SCAL = 2 * V6_NP * V6_NP * 4;
constexpr int V6_GP_IDX = V6_GP_SCAL + V6_NP * 16, V6_GP_BYTES = V6_GP_IDX + V6_NP * V6_NP;
constexpr int V6_OFF_GP = V6_STAGES * V6_STAGE_BYTES;
constexpr int V6_OFF_BAR = V6_OFF_GP + V6_GP_BYTES;
constexpr int V6_SMEM_BYTES = V6_OFF_BAR + (2 * V6_STAGES + 4 * V6_TBUF) * 8 + 16 + 1024;
// tensor memory, per buffer: S0q (-> O) | S0k (-> U) | Gram (-> R^T hi) | R^T lo
constexpr int V6_TM_COLS = 4 * V6_NP;
constexpr int V6_TM_SQ = 0, V6_TM_SK = V6_NP, V6_TM_D2 = 2 * V6_NP, V6_TM_RLO = 3 * V6_NP;
static_assert(V6_TBUF * V6_TM_COLS <= 512, "tensor memory");

// byte offset of element (row, col) inside an fp32 operand tile (two 128-byte-swizzled atoms)
__device__ __forceinline__ int v6_tile_off(int row, int col)
{
    return (col >> 5) * V6_ATOM + row * 128 + (((((col & 31) >> 2)) ^ (row & 7)) << 4) + ((col & 3) << 2);
}
// position of list entry d of node i
__device__ __forceinline__ int v6_at(int i, int d) { return ((d >> 2) * V6_NP + i) * 4 + (d & 3); }

}  // namespace

template <typename TOut>
__global__ void __launch_bounds__(V6_THREADS, 1)
verify_sm100_tc64_kernel(VerifyArgs a, int n_items, const __grid_constant__ CUtensorMap tmS0,
                         const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV)
{
    constexpr int NP = V6_NP;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + V6_OFF_BAR);
    uint64_t *empty = full + V6_STAGES;
    uint64_t *mma1_done = empty + V6_STAGES;
    uint64_t *ops_ready = mma1_done + V6_TBUF;
    uint64_t *mma2_done = ops_ready + V6_TBUF;
    uint64_t *tmem_free = mma2_done + V6_TBUF;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tmem_free + V6_TBUF);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < V6_STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int i = 0; i < V6_TBUF; ++i) {
            ptx::mbar_init(&mma1_done[i], 1);
            ptx::mbar_init(&ops_ready[i], V6_GROUP / 32);  // one arrival per warp
            ptx::mbar_init(&mma2_done[i], 1);
            ptx::mbar_init(&tmem_free[i], V6_GROUP / 32);
        }
        ptx::fence_barrier_init();
    }
    if (warp == V6_MMA1_WARP) {
        ptx::tmem_alloc(tmem_slot, 512);
        ptx::tmem_relinquish();
        ptx::tc_fence_before_sync();
    }
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    auto meta_mask = [&](unsigned char *stage) { return reinterpret_cast<unsigned long long *>(stage + V6_OFF_META); };
    auto meta_L = [&](unsigned char *stage) { return reinterpret_cast<float *>(stage + V6_OFF_META + NP * 8); };
    auto meta_beta = [&](unsigned char *stage) { return reinterpret_cast<float *>(stage + V6_OFF_META + NP * 12); };
    auto meta_nlo = [&](unsigned char *stage) { return reinterpret_cast<int *>(stage + V6_OFF_META + NP * 16); };

    if (warp >= V6_PROD_WARP0) {
        // ------------------------------------------------------------------ producer warp
        const int s = warp - V6_PROD_WARP0;
        unsigned char *stage = smem + s * V6_STAGE_BYTES;
        if (lane == 0) {
            ptx::prefetch_tmap(&tmS0), ptx::prefetch_tmap(&tmQ);
            ptx::prefetch_tmap(&tmK), ptx::prefetch_tmap(&tmV);
        }
        const int group = a.H_v / a.H_qk;
        // node scalars of an item, validated and loaded one round ahead (two nodes per lane)
        struct Pre {
            int item, b, h, lo, n, bad, flag;
            unsigned long long mk[2];
            float Lv[2], bv[2];
        };
        auto fetch = [&](int kk) {
            Pre p;
            p.item = blockIdx.x + kk * gridDim.x;
            p.b = 0, p.h = 0, p.lo = 0, p.n = 0, p.bad = 0, p.flag = 1;
            p.mk[0] = p.mk[1] = 0ull, p.Lv[0] = p.Lv[1] = 0.f, p.bv[0] = p.bv[1] = 0.f;
            if (p.item >= n_items) return p;
            p.b = p.item / a.H_v, p.h = p.item - p.b * a.H_v;
            p.lo = a.node_offsets[p.b];
            p.n = a.node_offsets[p.b + 1] - p.lo;
            if (p.n < 1 || p.n > a.max_nodes) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES;
                p.flag = a.cls_lo == 0;
            } else if (p.n <= a.cls_lo || p.n > a.cls_hi || p.n > NP) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES;  // another launch's size class: skipped, not flagged
                p.flag = 0;
            } else {
                int bp = 0;
                for (int i = lane; i < p.n; i += 32) {
                    const int par = a.parent[p.lo + i];
                    bp |= (par < -1 || par >= i);
                }
                if (__any_sync(0xffffffffu, bp)) p.bad = TREEWY_SEQ_BAD_PARENT;
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int i = lane + 32 * r;
                const bool on = !p.bad && i < p.n;
                p.mk[r] = on ? a.anc_mask[p.lo + i] : 0ull;
                p.Lv[r] = on ? a.cum_log_gate[(size_t)(p.lo + i) * a.H_v + p.h] : 0.f;
                p.bv[r] = on ? a.beta[(size_t)(p.lo + i) * a.H_v + p.h] : 0.f;
            }
            return p;
        };
        Pre cur = fetch(s);
        for (int kk = s;; kk += V6_STAGES) {
            if (cur.item >= n_items) break;
            const Pre p = cur;
            if (p.bad && p.flag && p.h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], p.bad);
            if (!ptx::mbar_wait(&empty[s], ((kk / V6_STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], TREEWY_SEQ_TIMEOUT);
                break;
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int i = lane + 32 * r;
                meta_mask(stage)[i] = p.mk[r], meta_L(stage)[i] = p.Lv[r], meta_beta(stage)[i] = p.bv[r];
            }
            if (lane == 0) meta_nlo(stage)[0] = p.bad ? 0 : p.n, meta_nlo(stage)[1] = p.lo;
            __syncwarp();
            if (lane == 0) {
                if (p.bad) {
                    ptx::mbar_arrive(&full[s]);
                } else {
                    ptx::mbar_arrive_expect_tx(&full[s], V6_TX_BYTES);
                    const int hq = p.h / group;
                    ptx::tma_load_2d(stage + V6_OFF_S0, &tmS0, 0, p.item * D, &full[s]);
                    ptx::tma_load_2d(stage + V6_OFF_S0 + V6_S0_HALF, &tmS0, 64, p.item * D, &full[s]);
                    ptx::tma_load_2d(stage, &tmQ, hq * D, p.lo, &full[s]);
                    ptx::tma_load_2d(stage + V6_QK_HALF, &tmQ, hq * D + 64, p.lo, &full[s]);
                    ptx::tma_load_2d(stage + NP * 128, &tmK, hq * D, p.lo, &full[s]);
                    ptx::tma_load_2d(stage + V6_QK_HALF + NP * 128, &tmK, hq * D + 64, p.lo, &full[s]);
                    ptx::tma_load_2d(stage + V6_OFF_V, &tmV, p.h * D, p.lo, &full[s]);
                }
            }
            cur = fetch(kk + V6_STAGES);  // in flight while this stage is being consumed
        }
    } else if (warp == V6_MMA1_WARP) {
        // ------------------------------------------------------------------ stage-1 MMAs
        //   D1[c, r] = sum_d S0[c,d] QK[r,d]   (N = 128: S0 q_i | S0 k_i)
        //   D2[r, j] = sum_d QK[r,d] K[j,d]    (rows: 64 q rows, 64 k rows; N = 64)
        constexpr uint32_t idesc1 = ptx::umma_idesc_bf16_f32(128, 2 * NP);
        constexpr uint32_t idesc2 = ptx::umma_idesc_bf16_f32(128, NP);
        for (int kk = 0;; ++kk) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int s = kk % V6_STAGES, buf = kk % V6_TBUF;
            unsigned char *stage = smem + s * V6_STAGE_BYTES;
            if (!ptx::mbar_wait(&full[s], (kk / V6_STAGES) & 1)) break;
            const int n = meta_nlo(stage)[0];
            if (!ptx::mbar_wait(&tmem_free[buf], ((kk / V6_TBUF) & 1) ^ 1)) break;
            ptx::tc_fence_after_sync();
            if (lane == 0) {
                if (n > 0) {
                    const uint32_t qk = ptx::smem_u32(stage), s0 = qk + V6_OFF_S0;
                    const uint32_t d1 = tmem_base + buf * V6_TM_COLS + V6_TM_SQ, d2 = tmem_base + buf * V6_TM_COLS + V6_TM_D2;
#pragma unroll 1
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t ko = (ks & 3) * 32;
                        ptx::umma_bf16(d1, ptx::umma_desc_k_sw128(s0 + (ks >> 2) * V6_S0_HALF + ko),
                                       ptx::umma_desc_k_sw128(qk + (ks >> 2) * V6_QK_HALF + ko), idesc1, ks > 0);
                    }
#pragma unroll 1
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t base = qk + (ks >> 2) * V6_QK_HALF + (ks & 3) * 32;
                        ptx::umma_bf16(d2, ptx::umma_desc_k_sw128(base), ptx::umma_desc_k_sw128(base + NP * 128),
                                       idesc2, ks > 0);
                    }
                    ptx::umma_commit(&mma1_done[buf]);
                } else {
                    ptx::mbar_arrive(&mma1_done[buf]);
                }
            }
            __syncwarp();
        }
    } else if (warp == V6_MMA2_WARP) {
        // ------------------------------------------------------------------ stage-2 MMAs
        //   U^T[c, i]  = sum_j R^T[c,j] T[i,j]                      (over the consumed S0 k columns)
        //   O^T[c, i] += sum_j R^T[c,j] W[i,j]   on top of g_i (S0 q_i)[c]
        // A = R^T from tensor memory (hi | lo), B = T / W tiles from shared memory; three passes
        // hi.hi + lo.hi + hi.lo each.
        constexpr uint32_t idesc = ptx::umma_idesc_tf32_f32(128, 2 * NP);
        for (int kk = 0;; ++kk) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int s = kk % V6_STAGES, buf = kk % V6_TBUF;
            unsigned char *stage = smem + s * V6_STAGE_BYTES;
            if (!ptx::mbar_wait(&ops_ready[buf], (kk / V6_TBUF) & 1)) break;
            ptx::tc_fence_after_sync();
            const int n = meta_nlo(stage)[0];
            if (lane == 0) {
                if (n > 0) {
                    const uint32_t base = ptx::smem_u32(stage);
                    const uint32_t tb = tmem_base + buf * V6_TM_COLS;
                    // three passes (hi.hi, lo.hi, hi.lo) of 8 steps of K = 8, accumulated on [g.S0q | 0]
#pragma unroll 1
                    for (int q = 0; q < 24; ++q) {
                        const int p = q >> 3, ks = q & 7;
                        const uint32_t ra = tb + (p == 1 ? V6_TM_RLO : V6_TM_D2) + ks * 8;
                        const uint32_t xb = base + (p == 2 ? V6_OFF_X_LO : V6_OFF_X_HI) + (ks >> 2) * V6_ATOM + (ks & 3) * 32;
                        ptx::umma_tf32_ts(tb + V6_TM_SQ, ra, ptx::umma_desc_k_sw128(xb), idesc, 1u);
                    }
                    ptx::umma_commit(&mma2_done[buf]);
                    ptx::umma_commit(&empty[s]);  // the stage's operand overlays have been consumed
                } else {
                    ptx::mbar_arrive(&mma2_done[buf]);
                    ptx::mbar_arrive(&empty[s]);
                }
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ consumer group
        const int t = tid;  // consumer warps are warps 0..3: thread t owns TMEM lane t
        unsigned char *gp = smem + V6_OFF_GP;
        float *Ap = reinterpret_cast<float *>(gp + V6_GP_AP);
        float *Pp = reinterpret_cast<float *>(gp + V6_GP_PP);
        float4 *scal = reinterpret_cast<float4 *>(gp + V6_GP_SCAL);
        unsigned char *idx = gp + V6_GP_IDX;
        TOut *Og = static_cast<TOut *>(a.O);
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const int rs = a.H_v * D;  // elements between a sequence's consecutive node rows

        int b_kk = -1, b_n = 0, b_lo = 0;  // the item whose back half (epilogue) is pending
        bool dead = false;
        for (int kk = 0; !dead; ++kk) {
            const int item = blockIdx.x + kk * gridDim.x;
            const bool have = item < n_items;
            int f_n = 0, f_lo = 0;
            if (have) {
                const int s = kk % V6_STAGES, buf = kk % V6_TBUF;
                unsigned char *stage = smem + s * V6_STAGE_BYTES;
                if (!ptx::mbar_wait(&mma1_done[buf], (kk / V6_TBUF) & 1)) {
                    if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                    dead = true;
                    break;
                }
                ptx::tc_fence_after_sync();
                ptx::mbar_wait(&full[s], (kk / V6_STAGES) & 1);  // already complete: acquires the meta block
                const int n = meta_nlo(stage)[0];
                const int lo = meta_nlo(stage)[1];
                const uint32_t tm = tmem_base + lane_base + buf * V6_TM_COLS;
                if (n > 0) {
                    const unsigned long long *mask = meta_mask(stage);
                    const float *Lm = meta_L(stage);
                    const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(stage + V6_OFF_V);
                    float *raw = reinterpret_cast<float *>(stage);  // over the dead [Q;K] / S0 tiles

                    // ---- G1: every thread's Gram row (q row of node t, or k row of node t - 64)
#pragma unroll 1
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        if (c0 < n) {
                            uint32_t g[16];
                            ptx::tmem_ld16(tm + V6_TM_D2 + c0, g);
                            ptx::tmem_wait_ld();
                            float4 *dst = reinterpret_cast<float4 *>(raw + t * V6_RLD + c0);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                dst[q] = make_float4(__uint_as_float(g[4 * q]), __uint_as_float(g[4 * q + 1]),
                                                     __uint_as_float(g[4 * q + 2]), __uint_as_float(g[4 * q + 3]));
                        }
                    }
                    ptx::named_sync(1, V6_GROUP);

                    // ---- G2: scaled ancestor lists; threads 0..63 build P[i][.], threads 64..127 A[i][.]
                    const int i = t & (NP - 1);
                    const bool a_kind = t >= NP;
                    const bool valid = i < n;
                    const unsigned long long mi = valid ? mask[i] : 0ull;
                    const int dp = valid ? __popcll(mi) - 1 : 0;  // ancestors of node i
                    const float Li = Lm[i];
                    const float bi = meta_beta(stage)[i];
                    {
                        const float scale = a_kind ? bi : 1.f;
                        const float *row = raw + t * V6_RLD;
                        unsigned long long m = mi & ~(1ull << i);
#pragma unroll 1
                        for (int d = 0; d < dp; d += 2) {  // two ancestors per round: independent chains
                            const int j0 = __ffsll((long long)m) - 1;
                            m &= m - 1;
                            const bool two = d + 1 < dp;
                            const int j1 = two ? __ffsll((long long)m) - 1 : j0;
                            m &= m - 1;
                            const float v0 = scale * __expf(Li - Lm[j0]) * row[j0];
                            const float v1 = scale * __expf(Li - Lm[j1]) * row[j1];
                            if (a_kind) {
                                Ap[v6_at(i, d)] = v0;
                                if (two) Ap[v6_at(i, d + 1)] = v1;
                            } else {
                                Pp[v6_at(i, d)] = v0, idx[v6_at(i, d)] = (unsigned char)j0;
                                if (two) Pp[v6_at(i, d + 1)] = v1, idx[v6_at(i, d + 1)] = (unsigned char)j1;
                            }
                        }
                        if (!a_kind && valid) {
                            const float gi = __expf(Li);
                            scal[i] = make_float4(bi, bi * gi, gi, row[i]);
                        }
                    }
                    // lists and scalars are in place, the raw rows are dead; learn whether any path is deep
                    const bool deep = ptx::named_sync_or(1, V6_GROUP, dp > 8);

                    // ---- T: row i of T = (I + A)^-1 (threads 64..127) and of W = P T (threads 0..63) by
                    // back-substitution along node i's root path j_0 .. j_{dp-1}, j_dp = i:
                    //   x_dp = 1 (T) or P[i][i] (W);  x_e = p_e - sum_{f > e} x_f A[j_f][j_e]
                    if (valid) {
                        const bool wrow = !a_kind;
                        const float top = wrow ? scal[i].w : 1.f;
                        unsigned char *Mhi = stage + (wrow ? V6_OFF_W_HI : V6_OFF_T_HI);
                        unsigned char *Mlo = stage + (wrow ? V6_OFF_W_LO : V6_OFF_T_LO);
#pragma unroll
                        for (int q = 0; q < 16; ++q) {  // the row starts as zeros
                            const int off = (q >> 3) * V6_ATOM + i * 128 + (((q & 7) ^ (i & 7)) << 4);  // bank-conflict free
                            *reinterpret_cast<uint4 *>(Mhi + off) = make_uint4(0u, 0u, 0u, 0u);
                            *reinterpret_cast<uint4 *>(Mlo + off) = make_uint4(0u, 0u, 0u, 0u);
                        }
                        if (!deep) {  // registers only; every load is unconditional (all addresses are
                                      // valid) and masked by a select, so the phase has no branches
                            int jf[9];
                            float x[9], pe[8], co[9][8];
#pragma unroll
                            for (int e = 0; e < 9; ++e) {
                                const int j = idx[v6_at(i, e < 8 ? e : 7)];
                                jf[e] = e < dp ? j : i;
                                x[e] = e == dp ? top : 0.f;
                            }
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const float pv = Pp[v6_at(i, e)];
                                pe[e] = (wrow && e < dp) ? pv : 0.f;
#pragma unroll
                                for (int f = e + 1; f < 9; ++f) {
                                    const float cv = Ap[v6_at(jf[f], e)];
                                    co[f][e] = f <= dp ? cv : 0.f;
                                }
                            }
#pragma unroll
                            for (int e = 7; e >= 0; --e) {
                                float acc = pe[e];
#pragma unroll
                                for (int f = e + 1; f < 9; ++f) acc = fmaf(-x[f], co[f][e], acc);
                                x[e] = e < dp ? acc : x[e];
                            }
                            // entries beyond the path all aim at the diagonal and carry 0; going down
                            // from e = 8 the real diagonal entry (e = dp) is written after them
#pragma unroll
                            for (int e = 8; e >= 0; --e) {
                                const float hi = ptx::tf32_hi(x[e]);
                                const int off = v6_tile_off(i, jf[e]);
                                *reinterpret_cast<float *>(Mhi + off) = hi;
                                *reinterpret_cast<float *>(Mlo + off) = x[e] - hi;
                            }
                        } else {  // deep paths: x_e is kept in the hi tile at its final column
                            *reinterpret_cast<float *>(Mhi + v6_tile_off(i, i)) = top;
#pragma unroll 1
                            for (int e = dp - 1; e >= 0; --e) {
                                float acc = wrow ? Pp[v6_at(i, e)] : 0.f;
#pragma unroll 1
                                for (int f = e + 1; f <= dp; ++f) {
                                    const int j = (f == dp) ? i : idx[v6_at(i, f)];
                                    acc = fmaf(-*reinterpret_cast<const float *>(Mhi + v6_tile_off(i, j)),
                                               Ap[v6_at(j, e)], acc);
                                }
                                *reinterpret_cast<float *>(Mhi + v6_tile_off(i, idx[v6_at(i, e)])) = acc;
                            }
#pragma unroll 1
                            for (int e = 0; e <= dp; ++e) {
                                const int off = v6_tile_off(i, (e == dp) ? i : idx[v6_at(i, e)]);
                                const float val = *reinterpret_cast<const float *>(Mhi + off), hi = ptx::tf32_hi(val);
                                *reinterpret_cast<float *>(Mhi + off) = hi;
                                *reinterpret_cast<float *>(Mlo + off) = val - hi;
                            }
                        }
                    }

                    // ---- R: row t of R^T, r_j = beta_j v_j - beta_j g_j (S0 k_j), hi | lo into tensor
                    // memory over the consumed Gram columns; then g_i (S0 q_i) in place
#pragma unroll 1
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        uint32_t hi[16], lo[16];
                        if (c0 < n) {
                            uint32_t sk[16];
                            ptx::tmem_ld16(tm + V6_TM_SK + c0, sk);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) {
                                const int j = c0 + jj;
                                const float4 sc = scal[j];
                                const float v = __bfloat162float(vs[j * D + t]);
                                const float val = j < n ? fmaf(-sc.y, __uint_as_float(sk[jj]), sc.x * v) : 0.f;
                                const float h = ptx::tf32_hi(val);
                                hi[jj] = __float_as_uint(h), lo[jj] = __float_as_uint(val - h);
                                sk[jj] = 0u;
                            }
                            ptx::tmem_st16(tm + V6_TM_SK + c0, sk);  // u_j accumulates on zeros
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) hi[jj] = 0u, lo[jj] = 0u;
                        }
                        ptx::tmem_st16(tm + V6_TM_D2 + c0, hi);
                        ptx::tmem_st16(tm + V6_TM_RLO + c0, lo);
                    }
#pragma unroll 1
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        if (c0 < n) {
                            uint32_t sq[16];
                            ptx::tmem_ld16(tm + V6_TM_SQ + c0, sq);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                sq[jj] = __float_as_uint(scal[c0 + jj].z * __uint_as_float(sq[jj]));
                            ptx::tmem_st16(tm + V6_TM_SQ + c0, sq);
                        }
                    }
                    ptx::tmem_wait_st();
                    ptx::fence_proxy_async();  // T / W tiles were written by ordinary stores
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&ops_ready[buf]);
                f_n = n, f_lo = lo;
            }

            if (b_kk >= 0) {
                // ---- back half of the previous item: u_i = DU[i], o_i = DO[i]
                const int pk = b_kk, n = b_n, lo = b_lo;
                const int pitem = blockIdx.x + pk * gridDim.x, h = pitem % a.H_v;
                const int buf = pk % V6_TBUF;
                const uint32_t tm = tmem_base + lane_base + buf * V6_TM_COLS;
                if (!ptx::mbar_wait(&mma2_done[buf], (pk / V6_TBUF) & 1)) {
                    if (t == 0 && a.seq_status) atomicOr(&a.seq_status[pitem / a.H_v], TREEWY_SEQ_TIMEOUT);
                    break;
                }
                ptx::tc_fence_after_sync();
                if (n > 0) {
                    float *Ub = a.U + ((size_t)lo * a.H_v + h) * D + t;
                    TOut *Ob = Og + ((size_t)lo * a.H_v + h) * D + t;
#pragma unroll 1
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        if (c0 < n) {
                            uint32_t du[16], dout[16];
                            ptx::tmem_ld16(tm + V6_TM_SK + c0, du);
                            ptx::tmem_ld16(tm + V6_TM_SQ + c0, dout);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) {
                                const int node = c0 + jj;
                                st_global_if(Ub + node * rs, __uint_as_float(du[jj]), node < n);
                                st_global_if(Ob + node * rs, __uint_as_float(dout[jj]), node < n);
                            }
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&tmem_free[buf]);
            }
            if (!have) break;
            b_kk = kk, b_n = f_n, b_lo = f_lo;
        }
    }

    // common exit: tensor memory goes back once every role is done with it
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == V6_MMA1_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

namespace {

template <typename TOut> cudaError_t launch_v6(const VerifyArgs &a, int T, cudaStream_t stream)
{
    const long long n_items = (long long)a.B * a.H_v;
    VerifyMaps m;
    if (!make_verify_maps(&m, a.S0, a.q, a.k, a.v, n_items, T, a.H_v, a.H_qk, V6_NP)) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(verify_sm100_tc64_kernel<TOut>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             V6_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    verify_sm100_tc64_kernel<TOut><<<grid, V6_THREADS, V6_SMEM_BYTES, stream>>>(a, (int)n_items, m.S0, m.Q, m.K,
                                                                                m.V);
    return cudaGetLastError();
}

}  // namespace

// trees of 33..64 nodes (the launch's size class), both contractions on the tensor cores
cudaError_t launch_verify_sm100_tc64(const VerifyArgs &a, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (od == TREEWY_F32) return launch_v6<float>(a, T, stream);
    return launch_v6<__nv_bfloat16>(a, T, stream);
}

}  // namespace treewy
