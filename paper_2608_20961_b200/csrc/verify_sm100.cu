// treewy_verify, bf16 production kernel for sm_100a (Section 3: Eq. 2 and the read-out).
//
// Persistent, warp-specialised, one CTA per SM; a work item is one (sequence b, value head h).
//
//   producer warps (one per shared-memory stage)
//       TMA tensor-map loads, 128-byte swizzle, all counted on the stage's mbarrier:
//       the 128x128 bf16 state tile S0[b,h] (two 64-column boxes), the sequence's q rows and
//       k rows stacked as [Q;K] (2*NP rows), its v rows; plus mask / log-gate / beta of the
//       nodes by ordinary loads.  Sequences are validated here (bad ones are skipped).
//   MMA warp (one elected thread issues tcgen05.mma, accumulators in tensor memory)
//       D1[c, r] = sum_d S0[c,d] * QK[r,d]      M = 128 (d_v), N = 2*NP, K = 128
//                  -> columns 0..NP-1 hold (S0 q_i)[c], columns NP.. hold (S0 k_i)[c]
//       D2[r, j] = sum_d QK[r,d] * K[j,d]        M = 128 (rows beyond 2*NP are don't-care),
//                  -> rows 0..NP-1 hold q_i.k_j, rows NP.. hold k_i.k_j      N = NP, K = 128
//       Both operands are K-major as stored, so nothing is transposed; bf16 products are
//       exact in fp32, only the fp32 accumulation rounds.  TMEM is double-buffered so the
//       MMAs of the next item run under the current item's solve.
//   consumer groups (128 threads each; thread c of a group owns TMEM lane c = row c of d_v;
//   groups take alternate items so one group's dependent chain hides under the other's)
//       phase G: thread r reads row r of D2 and scales + masks it, branch-free, into per-node
//           PATH lists kept in the stage's operand tiles (dead once the MMAs have completed):
//           A[i][d] = beta_i e^{L_i-L_j} k_i.k_j ,  P[i][d] = e^{L_i-L_j} q_i.k_j ,  idx[i][d] = j
//           for j the d-th ancestor of i (zero-padded to a multiple of four), plus
//           {beta_i, beta_i g_i, g_i, P[i][i]} per node;
//       phase N: every thread runs the forward substitution of (I + A) U = R for its own
//           column and reads the outputs out of the same pass:
//              u_i = beta_i v_i - beta_i g_i (S0 k_i) - sum_d A[i][d] u_{idx[i][d]} ,
//              o_i = g_i (S0 q_i) + sum_d P[i][d] u_{idx[i][d]} + P[i][i] u_i .
//           Nodes are taken in LEVEL order (sorted by depth): nodes of one depth do not depend
//           on each other and have equally long lists, so four of them are solved side by side
//           with all their loads in flight together (short levels repeat their first node,
//           which recomputes and rewrites identical values).  A single thread is latency
//           bound on this chain; the four-way batch is where its instruction-level
//           parallelism comes from.  tcgen05.ld (one run-time column per node) hands thread
//           c exactly (S0 q_i)[c] and (S0 k_i)[c], so no value crosses threads.  U (fp32) and
//           O are stored coalesced (a warp writes 128 contiguous bytes per node).
//
// Every mbarrier wait is bounded; on give-up the role leaves its loop, TREEWY_SEQ_TIMEOUT is
// raised, and the CTA still reaches the common exit where tensor memory is freed.
#include <cuda.h>

#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr int VS_GROUP = 128;  // threads of one consumer group
constexpr uint32_t VS_TMEM_COLS = 512;

template <int NP> struct VsCfg {
        static constexpr int GROUPS = NP <= 32 ? 2 : 1;
    static constexpr int STAGES = NP <= 16 ? 4 : (NP <= 32 ? 3 : 2);
    static constexpr int TBUF = GROUPS > 2 ? GROUPS : 2;  // TMEM accumulator buffers
    static constexpr int CONSUMERS = VS_GROUP * GROUPS;
    static constexpr int MMA_WARP = CONSUMERS / 32;
    static constexpr int THREADS = CONSUMERS + 32 + 32 * STAGES;
    static constexpr int QK_HALF = 2 * NP * 128;  // one 64-column half of the [Q;K] rows, bytes
    static constexpr int QK_BYTES = 2 * QK_HALF;
    static constexpr int S0_HALF = D * 128;
    static constexpr int S0_BYTES = 2 * S0_HALF;
    static constexpr int V_BYTES = NP * D * 2;
    static constexpr int OFF_S0 = QK_BYTES;
    static constexpr int OFF_V = OFF_S0 + S0_BYTES;
    static constexpr int OFF_META = OFF_V + V_BYTES;
    // mask u64, L f32, beta f32 per node; level order and its depths (bytes, 4 pad each); n, lo
    static constexpr int META_BYTES = NP * 16 + 2 * (NP + 4) + 16;
    static constexpr int STAGE_BYTES = (OFF_META + META_BYTES + 1023) / 1024 * 1024;
    // scratch inside a stage whose MMAs are done (operand tiles are dead by then)
    // path lists are stored [d / 4][node][d % 4]: a node's four consecutive ancestors form one
    // 16-byte (4-byte for indices) word, and neighbouring nodes are neighbouring words
    static constexpr int OFF_AP = OFF_S0;                // A path lists, NP*NP f32
    static constexpr int OFF_PP = OFF_S0 + NP * NP * 4;  // P path lists, NP*NP f32
    static constexpr int OFF_IDX = 0;                    // ancestor indices, NP*NP u8
    static constexpr int OFF_SCAL = NP * NP;             // {beta, beta g, g, P_ii} per node
    static_assert(2 * NP * NP * 4 <= S0_BYTES && OFF_SCAL + NP * 16 <= QK_BYTES, "scratch fits");
    static constexpr int OFF_US = STAGES * STAGE_BYTES;  // GROUPS x [NP][128] f32
    static constexpr int OFF_BAR = OFF_US + GROUPS * NP * D * 4;
    static constexpr int SMEM_BYTES = OFF_BAR + (2 * STAGES + 2 * TBUF) * 8 + 16 + 1024;  // + align slack
    static constexpr uint32_t TX_BYTES = S0_BYTES + QK_BYTES + V_BYTES;
};

struct VsMeta {  // view of a stage's meta block
    unsigned long long *mask;
    float *L, *beta;
    unsigned char *order;  // [NP+4] nodes sorted by (depth, index), padded with 0
    unsigned char *pdep;   // [NP+4] depth of order[p], padded with 255
    int *n_lo;
};
template <int NP> __device__ __forceinline__ VsMeta vs_meta(unsigned char *stage)
{
    unsigned char *m = stage + VsCfg<NP>::OFF_META;
    VsMeta r;
    r.mask = reinterpret_cast<unsigned long long *>(m);
    r.L = reinterpret_cast<float *>(m + NP * 8);
    r.beta = r.L + NP;
    r.n_lo = reinterpret_cast<int *>(r.beta + NP);
    r.order = reinterpret_cast<unsigned char *>(r.n_lo + 4);
    r.pdep = r.order + NP + 4;
    return r;
}

template <int NP, typename TOut>
__global__ void __launch_bounds__(VsCfg<NP>::THREADS, 1)
verify_sm100_kernel(VerifyArgs a, int n_items, const __grid_constant__ CUtensorMap tmS0,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV)
{
    using C = VsCfg<NP>;
    extern __shared__ unsigned char smem_dyn[];
    // 1024-byte phase for the swizzled operand tiles
    unsigned char *smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint64_t *empty = full + C::STAGES;
    uint64_t *mma_done = empty + C::STAGES;
    uint64_t *tmem_free = mma_done + C::TBUF;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tmem_free + C::TBUF);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int MMA_WARP = C::MMA_WARP;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], VS_GROUP);
        }
        for (int i = 0; i < C::TBUF; ++i) {
            ptx::mbar_init(&mma_done[i], 1);
            ptx::mbar_init(&tmem_free[i], VS_GROUP);
        }
        ptx::fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(tmem_slot, VS_TMEM_COLS);
        ptx::tmem_relinquish();
        ptx::tc_fence_before_sync();
    }
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp > MMA_WARP) {
        // ------------------------------------------------------------------ producer warp
        const int s = warp - MMA_WARP - 1;
        unsigned char *stage = smem + s * C::STAGE_BYTES;
        const VsMeta mt = vs_meta<NP>(stage);
        if (lane == 0) {
            ptx::prefetch_tmap(&tmS0), ptx::prefetch_tmap(&tmQ);
            ptx::prefetch_tmap(&tmK), ptx::prefetch_tmap(&tmV);
        }
        const int group = a.H_v / a.H_qk;
        for (int kk = s;; kk += C::STAGES) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int b = item / a.H_v, h = item - b * a.H_v;
            const int lo = a.node_offsets[b];
            const int n = a.node_offsets[b + 1] - lo;
            int bad = 0;
            bool other_class = false;  // handled by another launch: skipped here without a flag
            if (n < 1 || n > a.max_nodes) {
                bad = TREEWY_SEQ_TOO_MANY_NODES;
                other_class = a.cls_lo != 0;
            } else if (n <= a.cls_lo || n > a.cls_hi || n > NP) {
                bad = TREEWY_SEQ_TOO_MANY_NODES;
                other_class = true;
            } else {
                int bp = 0;
                for (int i = lane; i < n; i += 32) {
                    const int p = a.parent[lo + i];
                    bp |= (p < -1 || p >= i);
                }
                if (__any_sync(0xffffffffu, bp)) bad = TREEWY_SEQ_BAD_PARENT;
            }
            if (bad && !other_class && h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
            // node scalars: issued before the wait so their latency hides under it
            constexpr int R = (NP + 4 + 31) / 32;
            unsigned long long mk[R];
            float Lv[R], bv[R];
            int ord[R], pd[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int i = lane + 32 * r;
                const bool on = !bad && i < n;
                mk[r] = on ? a.anc_mask[lo + i] : 0ull;
                Lv[r] = on ? a.cum_log_gate[(size_t)(lo + i) * a.H_v + h] : 0.f;
                bv[r] = on ? a.beta[(size_t)(lo + i) * a.H_v + h] : 0.f;
                ord[r] = on ? min((int)a.level_order[lo + i], n - 1) : 0;
                pd[r] = on ? (a.depth[lo + ord[r]] & 63) : 255;
            }
            if (!ptx::mbar_wait(&empty[s], ((kk / C::STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], TREEWY_SEQ_TIMEOUT);
                break;
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int i = lane + 32 * r;
                if (i < NP) mt.mask[i] = mk[r], mt.L[i] = Lv[r], mt.beta[i] = bv[r];
                if (i < NP + 4) mt.order[i] = (unsigned char)ord[r], mt.pdep[i] = (unsigned char)pd[r];
            }
            if (lane == 0) mt.n_lo[0] = bad ? 0 : n, mt.n_lo[1] = lo;
            __syncwarp();
            if (lane == 0) {
                if (bad) {
                    ptx::mbar_arrive(&full[s]);
                } else {
                    ptx::mbar_arrive_expect_tx(&full[s], C::TX_BYTES);
                    const int hq = h / group;
                    ptx::tma_load_2d(stage + C::OFF_S0, &tmS0, 0, item * D, &full[s]);
                    ptx::tma_load_2d(stage + C::OFF_S0 + C::S0_HALF, &tmS0, 64, item * D, &full[s]);
                    ptx::tma_load_2d(stage, &tmQ, hq * D, lo, &full[s]);
                    ptx::tma_load_2d(stage + C::QK_HALF, &tmQ, hq * D + 64, lo, &full[s]);
                    ptx::tma_load_2d(stage + NP * 128, &tmK, hq * D, lo, &full[s]);
                    ptx::tma_load_2d(stage + C::QK_HALF + NP * 128, &tmK, hq * D + 64, lo, &full[s]);
                    ptx::tma_load_2d(stage + C::OFF_V, &tmV, h * D, lo, &full[s]);
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------------ MMA warp
        constexpr uint32_t idesc1 = ptx::umma_idesc_bf16_f32(128, 2 * NP);
        constexpr uint32_t idesc2 = ptx::umma_idesc_bf16_f32(128, NP);
        for (int kk = 0;; ++kk) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            if (!ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1)) break;
            const int n = vs_meta<NP>(stage).n_lo[0];
            if (!ptx::mbar_wait(&tmem_free[buf], ((kk / C::TBUF) & 1) ^ 1)) break;
            ptx::tc_fence_after_sync();
            if (lane == 0) {
                if (n > 0) {
                    const uint32_t qk = ptx::smem_u32(stage), s0 = qk + C::OFF_S0;
                    const uint32_t d1 = tmem_base + buf * 3 * NP, d2 = d1 + 2 * NP;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t ko = (ks & 3) * 32;
                        const uint64_t da = ptx::umma_desc_k_sw128(s0 + (ks >> 2) * C::S0_HALF + ko);
                        const uint64_t db = ptx::umma_desc_k_sw128(qk + (ks >> 2) * C::QK_HALF + ko);
                        ptx::umma_bf16(d1, da, db, idesc1, ks > 0);
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t ko = (ks & 3) * 32;
                        const uint32_t base = qk + (ks >> 2) * C::QK_HALF + ko;
                        const uint64_t da = ptx::umma_desc_k_sw128(base);
                        const uint64_t db = ptx::umma_desc_k_sw128(base + NP * 128);
                        ptx::umma_bf16(d2, da, db, idesc2, ks > 0);
                    }
                    ptx::umma_commit(&mma_done[buf]);
                } else {
                    ptx::mbar_arrive(&mma_done[buf]);
                }
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int grp = warp >> 2, t = tid & (VS_GROUP - 1);
        float *us = reinterpret_cast<float *>(smem + C::OFF_US) + grp * NP * D;
        for (int i = 0; i < NP; ++i) us[i * D + t] = 0.f;  // padded list entries read us[0]
        TOut *Og = static_cast<TOut *>(a.O);
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (int kk = grp;; kk += C::GROUPS) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            if (!ptx::mbar_wait(&mma_done[buf], (kk / C::TBUF) & 1)) {
                if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            ptx::tc_fence_after_sync();
            ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1);  // already complete: acquires the meta block
            const VsMeta mt = vs_meta<NP>(stage);
            const int n = mt.n_lo[0];
            if (n > 0) {
                const int lo = mt.n_lo[1];
                const int h = item % a.H_v;
                const uint32_t d1 = tmem_base + lane_base + buf * 3 * NP, d2 = d1 + 2 * NP;
                const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(stage + C::OFF_V);
                float *Ap = reinterpret_cast<float *>(stage + C::OFF_AP);
                float *Pp = reinterpret_cast<float *>(stage + C::OFF_PP);
                unsigned char *idx = stage + C::OFF_IDX;
                float4 *scal = reinterpret_cast<float4 *>(stage + C::OFF_SCAL);
                {   // phase G: Gram rows -> scaled path lists, without branches in the column scan
                    const bool p_row = t < n;                    // q_i . k_j, i = t
                    const bool a_row = t >= NP && t - NP < n;    // k_i . k_j, i = t - NP
                    const int i = p_row ? t : (a_row ? t - NP : 0);
                    const bool mine = p_row || a_row;
                    const unsigned long long mi = mine ? mt.mask[i] : 0ull;
                    const float Li = mt.L[i];
                    const float bi = mt.beta[i];
                    const float scale = a_row ? bi : 1.f;
                    float pself = 0.f;
                    int d = 0;  // ancestors of node i seen so far = list position of the next one
                    // a short rolled loop: the column scan runs once per item, so its code must
                    // stay small enough not to be refetched from L2 every time
                    for (int c0 = 0; c0 < n; c0 += 4) {
                        uint32_t g[4];
                        ptx::tmem_ld4(d2 + c0, g);
                        const uint32_t mc = (uint32_t)(mi >> c0);
                        const float4 Lj = *reinterpret_cast<const float4 *>(mt.L + c0);
                        ptx::tmem_wait_ld();
                        const float Ljs[4] = {Lj.x, Lj.y, Lj.z, Lj.w};
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            const bool on = (mc >> jj) & 1u;
                            const float e = __expf(on ? Li - Ljs[jj] : 0.f);
                            const float val = scale * e * __uint_as_float(g[jj]);
                            const bool self = (c0 + jj == i);
                            const int at = ((d >> 2) * NP + i) * 4 + (d & 3);
                            if (on && !self) {
                                if (p_row) Pp[at] = val, idx[at] = (unsigned char)(c0 + jj);
                                else Ap[at] = val;
                            }
                            pself = (on && self) ? val : pself;
                            d += (on && !self);
                        }
                    }
                    if (mine) {
                        const int lim = (d + 3) & ~3;
                        for (; d < lim; ++d) {
                            const int at = ((d >> 2) * NP + i) * 4 + (d & 3);
                            if (p_row) Pp[at] = 0.f, idx[at] = 0;
                            else Ap[at] = 0.f;
                        }
                        if (p_row) {
                            const float gi = __expf(Li);
                            scal[i] = make_float4(bi, bi * gi, gi, pself);
                        }
                    }
                }
                ptx::named_sync(1 + grp, VS_GROUP);

                // phase N: forward substitution + read-out, one column per thread, four
                // same-depth nodes per batch
                const float4 *Ap4 = reinterpret_cast<const float4 *>(Ap);
                const float4 *Pp4 = reinterpret_cast<const float4 *>(Pp);
                const uint32_t *idx4 = reinterpret_cast<const uint32_t *>(idx);
                float *Ub = a.U + ((size_t)lo * a.H_v + h) * D + t;
                TOut *Ob = Og + ((size_t)lo * a.H_v + h) * D + t;
                const int rs = a.H_v * D;  // elements between a sequence's consecutive node rows

                int pos = 0;
                while (pos < n) {
                    // the batch: up to four consecutive level-order entries of one depth
                    const int dep = mt.pdep[pos];
                    const bool c1 = mt.pdep[pos + 1] == dep;
                    const bool c2 = c1 && mt.pdep[pos + 2] == dep;
                    const bool c3 = c2 && mt.pdep[pos + 3] == dep;
                    int nb[4];
                    nb[0] = mt.order[pos];
                    nb[1] = c1 ? mt.order[pos + 1] : nb[0];
                    nb[2] = c2 ? mt.order[pos + 2] : nb[0];
                    nb[3] = c3 ? mt.order[pos + 3] : nb[0];
                    pos += 1 + c1 + c2 + c3;

                    uint32_t sq[4], sk[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        sq[x] = ptx::tmem_ld1(d1 + nb[x]);
                        sk[x] = ptx::tmem_ld1(d1 + NP + nb[x]);
                    }
                    float4 sc[4];
                    float vv[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        sc[x] = scal[nb[x]];
                        vv[x] = __bfloat162float(vs[nb[x] * D + t]);
                    }
                    ptx::tmem_wait_ld();
                    float ua[4], ub[4], oa[4], ob[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        ua[x] = fmaf(-sc[x].y, __uint_as_float(sk[x]), sc[x].x * vv[x]);
                        oa[x] = sc[x].z * __uint_as_float(sq[x]);
                        ub[x] = 0.f, ob[x] = 0.f;
                    }
                    for (int r4 = 0; r4 * 4 < dep; ++r4) {  // four ancestors per round, same count for the batch
                        uint32_t id[4];
                        float4 aa[4], pp[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            id[x] = idx4[r4 * NP + nb[x]];
                            aa[x] = Ap4[r4 * NP + nb[x]];
                            pp[x] = Pp4[r4 * NP + nb[x]];
                        }
                        float w[4][4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            w[x][0] = us[(id[x] & 255u) * D + t];
                            w[x][1] = us[((id[x] >> 8) & 255u) * D + t];
                            w[x][2] = us[((id[x] >> 16) & 255u) * D + t];
                            w[x][3] = us[(id[x] >> 24) * D + t];
                        }
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            ua[x] = fmaf(-aa[x].x, w[x][0], ua[x]), oa[x] = fmaf(pp[x].x, w[x][0], oa[x]);
                            ub[x] = fmaf(-aa[x].y, w[x][1], ub[x]), ob[x] = fmaf(pp[x].y, w[x][1], ob[x]);
                            ua[x] = fmaf(-aa[x].z, w[x][2], ua[x]), oa[x] = fmaf(pp[x].z, w[x][2], oa[x]);
                            ub[x] = fmaf(-aa[x].w, w[x][3], ub[x]), ob[x] = fmaf(pp[x].w, w[x][3], ob[x]);
                        }
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float u = ua[x] + ub[x];
                        const float o = fmaf(sc[x].w, u, oa[x] + ob[x]);
                        us[nb[x] * D + t] = u;
                        Ub[nb[x] * rs] = u;
                        Ob[nb[x] * rs] = from_f32<TOut>(o);
                    }
                }
                ptx::fence_proxy_async();  // scratch writes before the next TMA fill of this stage
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tmem_free[buf]);
            ptx::mbar_arrive(&empty[s]);
        }
    }

    // common exit: tensor memory goes back once every role is done with it
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, VS_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------ host side
namespace {

template <int NP, typename TOut>
cudaError_t launch_vs(const VerifyArgs &a, int T, cudaStream_t stream)
{
    using C = VsCfg<NP>;
    const long long n_items = (long long)a.B * a.H_v;
    VerifyMaps m;
    if (!make_verify_maps(&m, a.S0, a.q, a.k, a.v, n_items, T, a.H_v, a.H_qk, NP)) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(verify_sm100_kernel<NP, TOut>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    verify_sm100_kernel<NP, TOut><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(a, (int)n_items, m.S0, m.Q,
                                                                                m.K, m.V);
    return cudaGetLastError();
}

}  // namespace

// general variant: any tree of up to 64 nodes; the solve runs on the CUDA cores
cudaError_t launch_verify_sm100_simt(const VerifyArgs &a, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (od == TREEWY_F32) return launch_vs<64, float>(a, T, stream);
    return launch_vs<64, __nv_bfloat16>(a, T, stream);
}

}  // namespace treewy
