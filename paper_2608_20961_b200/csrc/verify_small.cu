// Verify (Eq. 2 and the read-out), and optionally the previous round's commit (Eq. 3) in front of
// it, for SMALL draft trees: up to 8 nodes per sequence, bf16 states.  This is the paper's production
// case (Section 4: a chain of a few multi-token-prediction drafts, verified and committed by one fused
// kernel); trees of up to 8 nodes take the same code, since a chain is the tree parent[i] = i - 1.
//
// With so few nodes the work per (sequence, head) is the 32 KiB state tile and little else, and the
// phases of one item are too short to be worth a warp role each (the kernel for larger trees hands
// an item from role to role seven times).  Here an item stays with ONE group of 128 threads from its
// first byte to its last, three groups per CTA work on three consecutive items side by side, and
// producer warps (one per stage of a four-stage ring) keep the tiles coming.
//
//   producer warp of stage s: validates the item, writes its scalars into the stage's meta block, and
//     issues the copies: state tile, q / k rows (64-column halves, 128-byte swizzle) and v rows by
//     TMA and -- fused mode -- the accepted path's k and u rows of the previous round by bulk copy;
//   group, per item:
//   * fused mode applies Eq. 3 to the tile in shared memory,
//     S[r][c] = g_a S[r][c] + sum_p u_p[r] (w_p k_p[c]), in the operation order of the commit
//     kernels (the stored state is bit-identical to theirs), rounds it to bf16 in place and sends
//     it back with a TMA store;
//   * S0 [Q;K]^T (M = 128 state rows, N = 16 = 8 q rows + 8 k rows, K = 128) and the Gram block
//     [Q;K] [Q;K]^T are sixteen tcgen05.mma from the tiles as they lie in shared memory, issued by
//     four threads into four accumulators each; the stage goes back to its producer as soon as the
//     tensor core has read it;
//   * sixteen lanes turn the Gram rows into A and P (Eq. 2); the 128 x 16 state product sits in
//     tensor memory with lane r = row r of the state, so thread r reads its S0 q_j and S0 k_j with
//     tcgen05.ld, solves its own column of (I + A) U = R by forward substitution in registers and
//     reads out o_j.
//
// (Earlier shapes, for the record.  S0 products with fp32 FMAs, thread r against row r: bound by
// the 128 bytes per clock that shared memory delivers to registers -- every thread re-reads every
// q / k vector -- at 2.8 us per tile and SM.  One CTA per item, four resident per SM: a chain of
// dependent latencies of 6 us per item that four CTAs do not hide.  Gram dot products on CUDA cores:
// 25 of 128 lanes busy for 2 k cycles, behind the MMA issue in the issuing warp.  Five stages and
// 544 threads: 96 registers per thread and the Eq. 3 pass spilled.)
#include <type_traits>

#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

namespace {

constexpr int VS_N = SMALL_MAX_NODES;
constexpr int VS_HALF = D * 128;            // bytes of one 64-column half of the state tile
constexpr int VS_QK_HALF = 2 * VS_N * 128;  // ... of the [Q;K] tile: 8 q rows, then 8 k rows
constexpr uint32_t VS_TMEM_COLS = 512;      // per group 128: four accumulators of 16 columns for S0 [Q;K]^T, four for the Gram block
static_assert(VS_N == 8, "the thread maps below are written for 8 nodes");

// what a stage says about its item (written by the producer warp)
struct VsMeta {
    int item;  // the item the stage holds or is being filled with (-1 before the first)
    int n;     // nodes to verify; 0 = nothing to verify (skipped or malformed sequence)
    int row;   // the item's first output row: (first packed node of the sequence) * H_v + head
    int srow;  // state tile: (state slot) * H_v + head
    int plen;  // fused mode: nodes on the accepted path of the previous round; -1 = nothing to commit
    float ga;  //             e^{L_a}
    uint32_t mask[VS_N];
    float L[VS_N], beta[VS_N];
    float w[VS_N];  // fused mode: e^{L_a - L_p} of the path nodes
};

template <bool FUSED> struct VsCfg {
    // (512 threads leave each 128 registers: the fused mode's Eq. 3 pass needs them)
    static constexpr int GROUPS = 3, STAGES = 4;
    static constexpr int PROD_WARP0 = GROUPS * 4;
    static constexpr int THREADS = GROUPS * 128 + STAGES * 32;
    // (the [Q;K] tile lies in front of the state tile: the Gram product reads 128 rows from its start,
    // the 112 past its own being whatever the state tile holds -- rows of the result nobody reads)
    static constexpr int OFF_QK = 0, OFF_TILE = 2 * VS_QK_HALF;
    static constexpr int OFF_V = OFF_TILE + 2 * VS_HALF;                 // v rows [8][128] bf16
    static constexpr int OFF_KP = OFF_V + VS_N * D * 2;                  // fused: k rows of the path [8][128] bf16
    static constexpr int OFF_UP = OFF_KP + (FUSED ? VS_N * D * 2 : 0);   //        u rows of the path [8][128] fp32
    static constexpr int STAGE_BYTES = (OFF_UP + (FUSED ? VS_N * D * 4 : 0) + 1023) / 1024 * 1024;
    static constexpr int OFF_META = STAGES * STAGE_BYTES;  // per stage: what the producer says about the item
    static constexpr int META_BYTES = ((int)sizeof(VsMeta) + 15) / 16 * 16;
    static constexpr int OFF_GRP = OFF_META + STAGES * META_BYTES;  // per group: what the read-out needs
    static constexpr int GRP_BYTES = (2 * VS_N * VS_N + 3 * VS_N) * 4;  // A, P, g_j, beta_j g_j, beta_j
    static constexpr int OFF_BAR = OFF_GRP + GROUPS * GRP_BYTES;
    static constexpr int SMEM_BYTES = OFF_BAR + (2 * STAGES + GROUPS) * 8 + 16 + 1024;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
};

template <typename TOut> __device__ __forceinline__ void store_out(TOut *p, float x);
template <> __device__ __forceinline__ void store_out<float>(float *p, float x) { *p = x; }
template <> __device__ __forceinline__ void store_out<__nv_bfloat16>(__nv_bfloat16 *p, float x)
{
    *p = __float2bfloat16_rn(x);
}

template <typename TOut, bool FUSED>
__global__ void __launch_bounds__(VsCfg<FUSED>::THREADS, 1)
verify_small_kernel(VerifyArgs a, PrevRound pv, int n_items, const __grid_constant__ CUtensorMap tmS0,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV)
{
    using C = VsCfg<FUSED>;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint64_t *empty = full + C::STAGES;
    uint64_t *mma_done = empty + C::STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(mma_done + C::GROUPS);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 4);  // one arrival per warp of the group that had the stage
        }
        for (int g = 0; g < C::GROUPS; ++g) ptx::mbar_init(&mma_done[g], 4);  // four issuing threads
        for (int s = 0; s < C::STAGES; ++s) reinterpret_cast<VsMeta *>(smem + C::OFF_META + s * C::META_BYTES)->item = -1;
        ptx::fence_barrier_init();
    }
    if (tid == 32) {  // (the descriptors are kernel parameters: fetched while the kernel before this one still runs)
        ptx::prefetch_tmap(&tmS0), ptx::prefetch_tmap(&tmQ);
        ptx::prefetch_tmap(&tmK), ptx::prefetch_tmap(&tmV);
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, VS_TMEM_COLS);
        ptx::tmem_relinquish();
        ptx::tc_fence_before_sync();
    }
    grid_dependency_wait();  // the kernel before this one on the stream has finished: global memory may be read
    if (tid == 0) ptx::wait_deadline_init(a.wait_cycles);
    __syncthreads();
    grid_dependency_trigger();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int group_heads = a.H_v / a.H_qk;

    if (warp >= C::PROD_WARP0) {
        // ------------------------------------------------------------------ producer warp of stage s
        const int s = warp - C::PROD_WARP0;
        unsigned char *stage = smem + s * C::STAGE_BYTES;
        // An item's scalars are validated and loaded one round ahead, so the dependent chain
        // node_offsets -> parent / mask / log-gate / beta never delays the issue of a copy.
        struct Pre {
            int item, b, h, lo, n, bad, flag, srow;
            uint32_t mk;  // lane i owns node i
            float Lv, bv;
            int plo, pbad, plen, pj;
            float La, wj;
        };
        auto fetch = [&](int kk) {
            Pre p;
            p.item = (int)blockIdx.x + kk * (int)gridDim.x;
            p.b = 0, p.h = 0, p.lo = 0, p.n = 0, p.bad = 0, p.flag = 1, p.srow = 0, p.mk = 0u, p.Lv = 0.f, p.bv = 0.f;
            p.plo = 0, p.pbad = 0, p.plen = -1, p.pj = 0, p.La = 0.f, p.wj = 0.f;
            if (p.item >= n_items) return p;
            p.b = p.item / a.H_v, p.h = p.item - p.b * a.H_v;
            p.lo = a.node_offsets[p.b];
            p.n = a.node_offsets[p.b + 1] - p.lo;
            const int slot = state_slot(a.state_index, a.n_states, p.b);
            p.srow = (slot < 0 ? 0 : slot) * a.H_v + p.h;
            if (slot < 0) {
                p.bad = TREEWY_SEQ_BAD_STATE, p.flag = a.cls_lo == 0;
            } else if (bad_offsets(p.lo, p.n, a.T)) {
                p.bad = TREEWY_SEQ_BAD_OFFSETS, p.flag = a.cls_lo == 0;
            } else if (p.n < 1 || p.n > a.max_nodes) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES, p.flag = a.cls_lo == 0;
            } else if (p.n <= a.cls_lo || p.n > a.cls_hi || p.n > VS_N) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES, p.flag = 0;  // another launch's size class: skipped, not flagged
            } else {
                const int par = lane < p.n ? a.parent[p.lo + lane] : -1;
                if (__any_sync(0xffffffffu, lane < p.n && (par < -1 || par >= lane))) p.bad = TREEWY_SEQ_BAD_PARENT;
            }
            if (!p.bad && lane < p.n) {
                p.mk = (uint32_t)a.anc_mask[p.lo + lane];
                p.Lv = a.cum_log_gate[(size_t)(p.lo + lane) * a.H_v + p.h];
                p.bv = a.beta[(size_t)(p.lo + lane) * a.H_v + p.h];
            }
            if constexpr (FUSED) {
                p.plo = pv.node_offsets[p.b];
                const int pn = pv.node_offsets[p.b + 1] - p.plo;
                const int acc = pv.accepted[p.b];
                if (slot < 0) {
                    p.pbad = TREEWY_SEQ_BAD_STATE;  // no state to commit into
                } else if (bad_offsets(p.plo, pn, pv.T)) {
                    p.pbad = TREEWY_SEQ_BAD_OFFSETS;
                } else if (pn < 1 || pn > pv.max_nodes || pn > VS_N) {
                    p.pbad = TREEWY_SEQ_TOO_MANY_NODES;
                } else {
                    const int par = lane < pn ? pv.parent[p.plo + lane] : -1;
                    if (__any_sync(0xffffffffu, lane < pn && (par < -1 || par >= lane))) p.pbad = TREEWY_SEQ_BAD_PARENT;
                    else if (acc < -1 || acc >= pn) p.pbad = TREEWY_SEQ_BAD_ACCEPTED;
                }
                if (!p.pbad && acc >= 0) {
                    const unsigned long long pmask = pv.anc_mask[p.plo + acc] & 0xffull;
                    p.La = pv.cum_log_gate[(size_t)(p.plo + acc) * a.H_v + p.h];
                    p.plen = __popcll(pmask);
                    if (lane < p.plen) {
                        p.pj = nth_set_bit(pmask, lane);
                        p.wj = expf(p.La - pv.cum_log_gate[(size_t)(p.plo + p.pj) * a.H_v + p.h]);
                    }
                }
            }
            return p;
        };
        // The first item of a stage: its state tile depends on nothing but the item's number, so it is put
        // in flight before the item's scalars are fetched.
        const int item0 = (int)blockIdx.x + s * (int)gridDim.x;
        const bool early = !a.state_index && item0 < n_items;
        if (early && lane == 0) {
            ptx::mbar_expect_tx(&full[s], 2 * VS_HALF);
            ptx::tma_load_2d(stage + C::OFF_TILE, &tmS0, 0, item0 * D, &full[s]);
            ptx::tma_load_2d(stage + C::OFF_TILE + VS_HALF, &tmS0, 64, item0 * D, &full[s]);
        }
        Pre cur = fetch(s);
#pragma unroll 1
        for (int kk = s;; kk += C::STAGES) {
            if (cur.item >= n_items) break;
            const Pre p = cur;
            if (lane == 0 && p.h == 0 && a.seq_status) {
                if (p.bad && p.flag) atomicOr(&a.seq_status[p.b], p.bad);
                if (FUSED && p.pbad) atomicOr(&a.seq_status[p.b], p.pbad);
            }
            if (!ptx::mbar_wait(&empty[s], ((kk / C::STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], TREEWY_SEQ_TIMEOUT);
                break;
            }
            VsMeta *meta = reinterpret_cast<VsMeta *>(smem + C::OFF_META + s * C::META_BYTES);
            if (lane < VS_N) meta->mask[lane] = p.mk, meta->L[lane] = p.Lv, meta->beta[lane] = p.bv, meta->w[lane] = p.wj;
            if (lane == 0) *reinterpret_cast<volatile int *>(&meta->item) = p.item;
            if (lane == 0) meta->n = p.bad ? 0 : p.n, meta->row = p.lo * a.H_v + p.h, meta->srow = p.srow, meta->plen = p.plen, meta->ga = expf(p.La);
            const int cnt = p.plen > 0 ? p.plen : 0;
            const bool need_tile = (!p.bad || p.plen >= 0) && !(early && kk == s);  // the state tile serves verify, commit or both
            const uint32_t tx = (need_tile ? 2 * VS_HALF : 0) + (p.bad ? 0 : 2 * VS_QK_HALF + VS_N * D * 2) + cnt * (D * 2 + D * 4);
            const int hq = p.h / group_heads;
            if (lane == 0 && need_tile) {
                ptx::tma_load_2d(stage + C::OFF_TILE, &tmS0, 0, p.srow * D, &full[s]);
                ptx::tma_load_2d(stage + C::OFF_TILE + VS_HALF, &tmS0, 64, p.srow * D, &full[s]);
            }
            if (lane == 0 && !p.bad) {  // rows lo .. lo + 7: those past the tree's end are never used
                ptx::tma_load_2d(stage + C::OFF_QK, &tmQ, hq * D, p.lo, &full[s]);
                ptx::tma_load_2d(stage + C::OFF_QK + VS_QK_HALF, &tmQ, hq * D + 64, p.lo, &full[s]);
                ptx::tma_load_2d(stage + C::OFF_QK + VS_N * 128, &tmK, hq * D, p.lo, &full[s]);
                ptx::tma_load_2d(stage + C::OFF_QK + VS_QK_HALF + VS_N * 128, &tmK, hq * D + 64, p.lo, &full[s]);
            }
            if (lane == 0 && !p.bad) ptx::tma_load_2d(stage + C::OFF_V, &tmV, p.h * D, p.lo, &full[s]);
            if constexpr (FUSED) {
                if (lane < cnt) {  // the accepted path's k and u rows of the previous round
                    const __nv_bfloat16 *kp = static_cast<const __nv_bfloat16 *>(pv.k);
                    ptx::bulk_g2s(stage + C::OFF_KP + lane * D * 2, kp + ((size_t)(p.plo + p.pj) * a.H_qk + hq) * D, D * 2,
                                  &full[s]);
                    ptx::bulk_g2s(stage + C::OFF_UP + lane * D * 4, pv.U + ((size_t)(p.plo + p.pj) * a.H_v + p.h) * D,
                                  D * 4, &full[s]);
                }
            }
            __syncwarp();  // the meta block is written, the copies are issued: announce them
            if (lane == 0) {
                if (tx == 0) ptx::mbar_arrive(&full[s]);
                else ptx::mbar_arrive_expect_tx(&full[s], tx);
            }
            cur = fetch(kk + C::STAGES);  // in flight while this stage is being consumed
        }
    } else {
        // ------------------------------------------------------------------ group g: items g, g + 3, ...
        const int g = warp >> 2, t = tid & 127;
        float *Am = reinterpret_cast<float *>(smem + C::OFF_GRP + g * C::GRP_BYTES), *Pm = Am + VS_N * VS_N, *Gm = Pm + VS_N * VS_N;
        const uint32_t tm = tmem_base + 128 * g;
        const int bar_id = 1 + g;
        uint32_t mma_phase = 0;
#pragma unroll 1
        for (int kk = g;; kk += C::GROUPS) {
            const int item = (int)blockIdx.x + kk * (int)gridDim.x;
            if (item >= n_items) break;
            const int s = kk % C::STAGES;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            const VsMeta *meta = reinterpret_cast<const VsMeta *>(smem + C::OFF_META + s * C::META_BYTES);
            // A stage is handed from group to group, so this group has not itself seen the stage's previous
            // phase complete, and a parity wait is only meaningful within one phase of the barrier's
            // current one.  The producer therefore names the item in the meta block before it fills the
            // stage: once that name is this item, the barrier is in this item's phase or past it.
            bool ready = true;
            {
                const volatile int *named = &meta->item;
                while (*named != item) {
                    if (ptx::wait_deadline_passed()) {
                        ready = false;
                        break;
                    }
                    __nanosleep(100);
                }
            }
            ready = ready && ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1);
            // (a barrier of the group: the outcome of the bounded wait is the same in all its threads,
            // and nobody is still in the previous item's read-out when A and P are rewritten)
            if (ptx::named_sync_or(bar_id, 128, !ready)) {
                if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            const int n = meta->n, row0 = meta->row, srow = meta->srow;
            const int plen = FUSED ? meta->plen : -1;
            if constexpr (FUSED) {
                if (plen >= 0) {
                    // Eq. 3 on the tile: thread (r0, cc) takes the 16-byte chunk cc of rows r0, r0 + 8, ...
                    const int cc = t & 15, r0 = t >> 4;
                    const float ga = meta->ga;
                    // (w_p k_p of the first four path nodes in registers; a longer path re-reads the rest
                    // from the stage for every row: rare, and it keeps the registers for three groups)
                    float kwr[4][8];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        if (p < plen) {
                            widen8(*reinterpret_cast<const uint4 *>(stage + C::OFF_KP + p * D * 2 + cc * 16), kwr[p]);
                            const float w = meta->w[p];
#pragma unroll
                            for (int e = 0; e < 8; ++e) kwr[p][e] *= w;
                        }
                    }
                    const float *up = reinterpret_cast<const float *>(stage + C::OFF_UP);
                    // (row r0 + 8 it has r & 7 = r0: the chunk sits at the same swizzled place in every row)
                    unsigned char *base = stage + C::OFF_TILE + (cc >> 3) * VS_HALF + r0 * 128 + (((cc & 7) ^ r0) << 4);
                    // (the round's code is compiled once per path length up to four: a path of one node
                    // then issues a quarter of the FMAs, not all of them predicated off)
                    auto pass = [&](auto ptag) {
                        constexpr int P = decltype(ptag)::value;
#pragma unroll 1
                        for (int it = 0; it < 16; it += 2) {
                            // two rows per round, every load ahead of the stores (which the compiler must
                            // otherwise assume to alias the u rows)
                            uint4 *px0 = reinterpret_cast<uint4 *>(base + it * 1024), *px1 = px0 + 64;
                            const int r = r0 + 8 * it;
                            float s0v[8], s1v[8], u0[P > 0 ? P : 1], u1[P > 0 ? P : 1];
                            widen8(*px0, s0v);
                            widen8(*px1, s1v);
#pragma unroll
                            for (int p = 0; p < P; ++p) u0[p] = up[p * D + r], u1[p] = up[p * D + r + 8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) s0v[e] *= ga, s1v[e] *= ga;
#pragma unroll
                            for (int p = 0; p < P; ++p) {
#pragma unroll
                                for (int e = 0; e < 8; ++e) s0v[e] = fmaf(u0[p], kwr[p][e], s0v[e]), s1v[e] = fmaf(u1[p], kwr[p][e], s1v[e]);
                            }
                            if constexpr (P == 4) {
#pragma unroll 1
                                for (int p = 4; p < plen; ++p) {
                                    float kx[8];
                                    widen8(*reinterpret_cast<const uint4 *>(stage + C::OFF_KP + p * D * 2 + cc * 16), kx);
                                    const float w = meta->w[p], ua = up[p * D + r], ub = up[p * D + r + 8];
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        const float kwv = kx[e] * w;
                                        s0v[e] = fmaf(ua, kwv, s0v[e]), s1v[e] = fmaf(ub, kwv, s1v[e]);
                                    }
                                }
                            }
                            uint4 y0, y1;
                            y0.x = pack_bf16(s0v[0], s0v[1]), y0.y = pack_bf16(s0v[2], s0v[3]);
                            y0.z = pack_bf16(s0v[4], s0v[5]), y0.w = pack_bf16(s0v[6], s0v[7]);
                            y1.x = pack_bf16(s1v[0], s1v[1]), y1.y = pack_bf16(s1v[2], s1v[3]);
                            y1.z = pack_bf16(s1v[4], s1v[5]), y1.w = pack_bf16(s1v[6], s1v[7]);
                            *px0 = y0, *px1 = y1;
                        }
                    };
                    switch (plen < 4 ? plen : 4) {
                    case 0: pass(std::integral_constant<int, 0>{}); break;
                    case 1: pass(std::integral_constant<int, 1>{}); break;
                    case 2: pass(std::integral_constant<int, 2>{}); break;
                    case 3: pass(std::integral_constant<int, 3>{}); break;
                    default: pass(std::integral_constant<int, 4>{}); break;
                    }
                    ptx::fence_proxy_async();  // written by ordinary stores, read by the TMA store and the tensor core
                }
            }
            if (plen >= 0) {  // the tile was rewritten by the whole group: a barrier before it is read
                ptx::tc_fence_before_sync();
                ptx::named_sync(bar_id, 128);
            }
            if (t == 0 && plen >= 0) {
                ptx::tma_store_2d(&tmS0, 0, srow * D, stage + C::OFF_TILE);
                ptx::tma_store_2d(&tmS0, 64, srow * D, stage + C::OFF_TILE + VS_HALF);
                ptx::bulk_commit_group();
            }
            if (n > 0 && (t & 31) == 0) {
                // [SQ | SK] = S0 [Q;K]^T (K = 128 in eight steps of 16) and the Gram block [Q;K] [Q;K]^T the
                // same way: rows 0..7 of that are q_j . (q_i | k_i), rows 8..15 are k_j . (q_i | k_i); its A
                // operand is read as 128 rows, of which only the first 16 are the tile's own (see VsCfg).
                // An MMA keeps its issuing thread for ~170 cycles, and MMAs into one accumulator run one
                // after the other (~450 cycles each at this size): so four threads issue four steps each,
                // every step pair into an accumulator of its own, and the read-out adds the four up.
                ptx::tc_fence_after_sync();
                constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(128, 2 * VS_N);
                const uint32_t s0 = ptx::smem_u32(stage + C::OFF_TILE), qk = ptx::smem_u32(stage + C::OFF_QK);
                const int w4 = t >> 5;            // 0, 1: state product; 2, 3: Gram block
                const int c0 = (w4 & 1) * 2;      // this thread's two accumulators
#pragma unroll 1
                for (int q = 0; q < 4; ++q) {
                    const int ks = (q >> 1) * 4 + c0 + (q & 1);  // steps c0, c0 + 1, then 4 + c0, 4 + c0 + 1
                    const uint64_t dq = ptx::umma_desc_k_sw128(qk + (ks >> 2) * VS_QK_HALF + (ks & 3) * 32);
                    if (w4 < 2)
                        ptx::umma_bf16(tm + 16 * (ks & 3), ptx::umma_desc_k_sw128(s0 + (ks >> 2) * VS_HALF + (ks & 3) * 32), dq,
                                       idesc, q >= 2);
                    else
                        ptx::umma_bf16(tm + 64 + 16 * (ks & 3), dq, dq, idesc, q >= 2);
                }
                ptx::umma_commit(&mma_done[g]);
            }
            if (n > 0) {
                const bool mma_ok = ptx::mbar_wait(&mma_done[g], mma_phase);
                mma_phase ^= 1u;
                // what the read-out needs of the stage goes to registers: the stage is handed back before it
                float vreg[VS_N] = {};
                {
                    const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(stage + C::OFF_V) + t;
#pragma unroll
                    for (int j = 0; j < VS_N; ++j)
                        if (j < n) vreg[j] = __bfloat162float(vs[j * D]);
                }
                uint32_t mj = 0u;   // threads 0..15: node j's ancestor-or-self mask
                float Lrow = 0.f, brow = 0.f, Lall[VS_N] = {};
                if (t < 2 * VS_N) {
                    mj = meta->mask[t & 7], Lrow = meta->L[t & 7], brow = meta->beta[t & 7];
#pragma unroll
                    for (int i = 0; i < VS_N; ++i) Lall[i] = meta->L[i];
                }
                if (ptx::named_sync_or(bar_id, 128, !mma_ok)) {
                    if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                    break;
                }
                // the stage goes back to its producer: the tensor core and every thread have read it
                if (t == 0 && plen >= 0) ptx::bulk_wait_group_read<0>();  // ... and so has the store
                ptx::mbar_arrive_warp(&empty[s]);
                ptx::tc_fence_after_sync();
                if (warp == 4 * g) {
                    // Gram rows -> A and P (Eq. 2): lane j < 8 holds q_j . k_i, lane 8 + j holds k_j . k_i
                    // in columns 8..15 of its row
                    uint32_t g0[16], g1[16], g2[16], g3[16];
                    ptx::tmem_ld16(tm + 64, g0), ptx::tmem_ld16(tm + 80, g1);
                    ptx::tmem_ld16(tm + 96, g2), ptx::tmem_ld16(tm + 112, g3);
                    ptx::tmem_wait_ld();
                    if (t < 2 * VS_N) {
                        const int j = t & 7;
                        const bool krow = t >= VS_N;  // k_j . k_i -> A (proper ancestors), q_j . k_i -> P (ancestor or self)
#pragma unroll
                        for (int i = 0; i < VS_N; ++i) {
                            const float dot = (__uint_as_float(g0[8 + i]) + __uint_as_float(g1[8 + i])) +
                                              (__uint_as_float(g2[8 + i]) + __uint_as_float(g3[8 + i]));
                            const bool on = j < n && i <= j && ((mj >> i) & 1u) && (!krow || i < j);
                            float val = on ? __expf(Lrow - Lall[i]) * dot : 0.f;
                            if (krow) val *= brow;
                            (krow ? Am : Pm)[j * VS_N + i] = val;
                        }
                        const float gj = __expf(Lrow);
                        if (krow) Gm[VS_N + j] = brow * gj, Gm[2 * VS_N + j] = brow;
                        else Gm[j] = gj;
                    }
                }
                ptx::named_sync(bar_id, 128);  // A and P are written
                // element t of r_j, u_j (forward substitution: parents come before children), o_j
                float d[16];
                {
                    uint32_t d0[16], d1[16], d2[16], d3[16];
                    const uint32_t tl = tm + ((uint32_t)((warp & 3) * 32) << 16);
                    ptx::tmem_ld16(tl, d0), ptx::tmem_ld16(tl + 16, d1);
                    ptx::tmem_ld16(tl + 32, d2), ptx::tmem_ld16(tl + 48, d3);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        d[c] = (__uint_as_float(d0[c]) + __uint_as_float(d1[c])) + (__uint_as_float(d2[c]) + __uint_as_float(d3[c]));
                }
                ptx::tc_fence_before_sync();
                float u[VS_N];
                const size_t urow = (size_t)row0 * D + t;
                TOut *Og = static_cast<TOut *>(a.O) + urow;
                const size_t rs = (size_t)a.H_v * D;
#pragma unroll
                for (int j = 0; j < VS_N; ++j) {
                    u[j] = 0.f;
                    if (j < n) {
                        float x = fmaf(-Gm[VS_N + j], d[VS_N + j], Gm[2 * VS_N + j] * vreg[j]);
                        float o = Gm[j] * d[j];
#pragma unroll
                        for (int i = 0; i < j; ++i) x = fmaf(-Am[j * VS_N + i], u[i], x);
                        u[j] = x;
#pragma unroll
                        for (int i = 0; i <= j; ++i) o = fmaf(Pm[j * VS_N + i], u[i], o);
                        store_u(a.U, urow + j * rs, x, a.u_half);
                        store_out(Og + j * rs, o);
                    }
                }
            }
            if (n == 0) {  // nothing verified: the stage goes back here
                if (t == 0 && plen >= 0) ptx::bulk_wait_group_read<0>();  // the store has read the tile
                ptx::mbar_arrive_warp(&empty[s]);
            }
        }
        if (t == 0) ptx::bulk_wait_group<0>();
    }

    // common exit: tensor memory goes back once every group is done with it
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, VS_TMEM_COLS);
    }
}

template <typename TOut, bool FUSED>
cudaError_t launch_vs(const VerifyArgs &a, const PrevRound &pv, int T, cudaStream_t stream)
{
    const long long n_items = (long long)a.B * a.H_v;
    const long long n_tiles = a.state_index ? (long long)a.n_states * a.H_v : n_items;
    VerifyMaps m;
    if (!make_verify_maps(&m, a.S0, a.q, a.k, a.v, n_tiles, T, a.H_v, a.H_qk, VS_N)) return cudaErrorInvalidValue;
    using C = VsCfg<FUSED>;
    int dev = 0, sms = 0;
    cudaError_t e = current_device_sms(&dev, &sms);
    if (e != cudaSuccess) return e;
    e = ensure_dynamic_smem(reinterpret_cast<const void *>(verify_small_kernel<TOut, FUSED>), C::SMEM_BYTES, dev);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    return launch_dependent(verify_small_kernel<TOut, FUSED>, dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, stream, a, pv,
                            (int)n_items, m.S0, m.Q, m.K, m.V);
}

}  // namespace

cudaError_t launch_verify_small(const VerifyArgs &a, const PrevRound *pv, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0 || T == 0) return cudaSuccess;
    const PrevRound none = {};
    if (pv)
        return od == TREEWY_F32 ? launch_vs<float, true>(a, *pv, T, stream) : launch_vs<__nv_bfloat16, true>(a, *pv, T, stream);
    return od == TREEWY_F32 ? launch_vs<float, false>(a, none, T, stream) : launch_vs<__nv_bfloat16, false>(a, none, T, stream);
}

}  // namespace treewy
