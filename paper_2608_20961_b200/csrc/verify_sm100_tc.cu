// treewy_verify, bf16 production kernel for trees of up to 32 nodes (Section 3: Eq. 2 and the
// read-out), with BOTH contractions of the method on the tcgen05 tensor cores:
//
//   stage 1 (bf16 x bf16 -> fp32):   D1 = S0 [Q;K]^T  (S0 q_i, S0 k_i),   D2 = [Q;K] K^T  (Gram)
//   stage 2 (bf16 x bf16 -> fp32, two-term operand splits):   [O | U]^T = [g.S0q | 0]^T + R^T [W;T]^T
//
// where R[j] = beta_j (v_j - g_j S0 k_j) is the right-hand side of Eq. 2, T = (I + A)^{-1} and
// W = P T.  The triangular system is not solved column by column: because A only couples a
// node with its ancestors, row i of T (and of W) lives on node i's root path and is the last
// row of the inverse of the small path matrix I + A_path, which one thread obtains by a
// back-substitution of depth(i) steps.  All rows are independent, so the sequential part of
// the solve shrinks from N steps per column to depth steps per node, done once per item, and
// the N x N x 128 products go to the tensor pipe.
//
// Accuracy of stage 2: every fp32 operand x is split as hi = bf16(x) and lo = bf16(x - hi), which
// leaves 2^-18 |x|; the kernel accumulates hi.hi + lo.hi + hi.lo in fp32 and drops lo.lo, so a
// product is off by at most 3 * 2^-18 of its size (three orders of magnitude below the bf16 rounding
// of O and of the committed state).  Against the same split on the tf32 pipe (2^-22, K = 8 per
// instruction, 4-byte operands) this halves the MMAs, the B tiles and the R^T columns in tensor memory.
//
// Roles (persistent CTA, one per SM; item = one (sequence, value head)).  Every phase of an item
// has its own warps and every role walks all items in order, so the per-item cost is that of the
// slowest role, not their sum; rings of buffers (4 load stages, 5 + 3 tensor-memory blocks, 2 slots
// for lists / scalars / v rows) let consecutive items overlap:
//   producer warps   TMA tensor-map loads of S0 and [Q;K] into a stage ring; node scalars and the
//                    path lists (index and gate ratio of every node's first 8 ancestors)
//   state-tile warp  (64-node instance) the S0 tiles have a ring of their own, shorter-lived than
//                    the stages, filled in item order by this warp
//   MMA-1 warp       stage-1 MMAs: SQ | SK into a block of the first TMEM ring, the Gram block
//                    into a block of the second                            -> mma1_done
//   Gram warps       Gram rows -> stash -> scaled ancestor lists (A, P), per-node scalars; zero the
//                    stage-2 B tiles (they overlay the dead [Q;K] tile)    -> lists_ready
//   solver warps     per-node back-substitution -> rows of T and W, scattered (hi, lo) into the
//                    swizzled B tiles; they also keep the v rows coming    -> ops_ready
//   R^T warps        (thread c = TMEM lane c = row c of d_v) row c of R^T as hi / lo back into
//                    tensor memory over the Gram block, g.S0q in place, zeros over S0k
//                                                                          -> ops_ready
//   MMA-2 warp       stage-2 MMAs, A = R^T from tensor memory (bf16 pairs), B = [W;T] from shared memory,
//                    three passes (hi.hi, lo.hi, hi.lo) accumulated on [g.S0q | 0]: [O | U]
//                                                                          -> mma2_done, stage and
//                                                                             R^T block released
//   epilogue warps   o_i and u_i leave tensor memory: coalesced stores     -> block released
//
// The kernel's code has to stay small: with this many roles in flight it was instruction-cache
// bound (a third of the instruction fetches missed) until the long loops were rolled and the slow
// path of the waits went out of line.
//
// Every mbarrier wait is bounded by one deadline per kernel; once it has passed, every role's next
// wait fails at once, the role leaves its loop, TREEWY_SEQ_TIMEOUT is raised, and the CTA still
// reaches the common exit where tensor memory is freed.
#include <cuda.h>

#include <type_traits>

#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr uint32_t VT_TMEM_COLS = 512;

template <int NP, bool FUSED> struct VtCfg {
    static_assert(NP == 16 || NP == 32 || (NP == 64 && !FUSED), "up to 64 nodes; the fused mode up to 32");
    static constexpr bool BIG = NP == 64;  // 33..64 nodes: shared memory and tensor memory hold three items
    // 64 nodes: the S0 tiles are not part of the stages but a ring of their own, S0_SLOTS deep, filled by
    // a warp of its own in item order.  A state tile lives from its copy to the end of stage 1, half as
    // long as the [Q;K] tile and what overlays it, so two tiles serve three stages.
    static constexpr bool S0_RING = BIG;
    static constexpr int S0_SLOTS = 2;
    static constexpr int NPL = (NP + 31) / 32;  // nodes per producer lane
    static constexpr int SLOTS = 2;  // list / scalar / v-row buffers alternate between consecutive items
    static constexpr int STAGES = BIG ? 3 : (FUSED ? 3 : 4) + (NP == 16 ? 1 : 0);  // as many as shared memory holds
    static constexpr int CGROUP = FUSED ? 128 : 0;  // threads of the commit group (fused mode)
    // (fused mode gives 128 columns of tensor memory to the commit's accumulator)
        static constexpr int TBUF = BIG ? 3 : FUSED ? 4 : 5;  // [SQ | SK] -> [O | U] blocks: held from stage 1 to the epilogue
    static constexpr int RBUF = BIG ? 2 : FUSED ? 2 : 3;  // [D2 | -] -> R^T (hi | lo) blocks: held from stage 1 to the end of stage 2
    // every phase of an item has its own warps, and every role walks all items in order
    // (64 nodes: two R^T groups, each taking half of the columns of every item)
    static constexpr int R_GROUPS = BIG ? 2 : 1;
    static constexpr int G_THREADS = BIG ? 128 : 64, T_THREADS = BIG ? 128 : 64, R_THREADS = 128 * R_GROUPS;
    static constexpr int E_THREADS = 128;
    static constexpr int G_WARP0 = 0, T_WARP0 = G_THREADS / 32, R_WARP0 = T_WARP0 + T_THREADS / 32;
    static constexpr int E_WARP0 = R_WARP0 + R_THREADS / 32;  // Gram (when 4 warps) / R / E: warp % 4 = TMEM lane quarter
    static constexpr int COMMIT_WARP0 = E_WARP0 + 4;
    static constexpr int MMA1_WARP = COMMIT_WARP0 + CGROUP / 32;
    static constexpr int MMA1B_WARP = MMA1_WARP + 1;  // the Gram chain of stage 1 has its own issuing warp
    static constexpr int MMA2_WARP = MMA1B_WARP + 1;
    static constexpr int PROD_WARP0 = MMA2_WARP + 1;
    static constexpr int S0P_WARP = PROD_WARP0 + STAGES;  // (S0_RING) the warp that fills the ring of S0 tiles
    static constexpr int THREADS = COMMIT_WARP0 * 32 + CGROUP + 96 + 32 * STAGES + (S0_RING ? 32 : 0);
    // stage: [Q;K] tile | S0 tile | (fused: previous round's path rows of k and U) | meta | (fused: path meta)
    // (the v rows go to the slots below, two items ahead)
    static constexpr int QK_HALF = 2 * NP * 128;
    static constexpr int QK_BYTES = 2 * QK_HALF;
    static constexpr int S0_HALF = D * 128;
    static constexpr int S0_BYTES = 2 * S0_HALF;
    static constexpr int OFF_S0 = QK_BYTES;  // (not S0_RING)
    static constexpr int PCH = 8;  // previous-round path nodes staged per item (fused mode)
    static constexpr int OFF_KP = OFF_S0 + S0_BYTES, OFF_UP = OFF_KP + PCH * D * 2;
    static constexpr int OFF_META = FUSED ? OFF_UP + PCH * D * 4 : S0_RING ? QK_BYTES : OFF_S0 + S0_BYTES;
    // mask u64, L f32, beta f32 per node; n, lo, deep; then the producer-built path lists of the
    // first 8 ancestors of every node: gate ratios e^{L_i - L_j} as [d / 4][node][d % 4] floats and
    // the ancestors' indices as [d / 4][node] words of four bytes
    static constexpr int META_RAT = NP * 16 + 16, META_IDX = META_RAT + 2 * NP * 16;
    static constexpr int META_BYTES = META_IDX + 2 * NP * 4;
    // 64 nodes: the meta blocks are not part of the stage but a ring of their own, twice as deep, so that
    // the producer writes an item's block (the path lists are 4 k cycles of one warp's time) while the
    // stage is still busy with the item before, not after it has been handed back.  (The fused mode has
    // room for such a ring too; it was tried and changed nothing there: its loads take as long as its lists.)
    static constexpr bool META_RING = BIG;
    static constexpr int OFF_PMETA = OFF_META + (META_RING ? 0 : META_BYTES);  // PathMeta of the previous round's commit
    static constexpr int META_SLOTS = META_RING ? 2 * STAGES : STAGES, META_STRIDE = (META_BYTES + 15) / 16 * 16;
    static constexpr int STAGE_BYTES = (OFF_PMETA + (FUSED ? 128 : 0) + 1023) / 1024 * 1024;
    // stage-2 B operand [W;T]: 2 NP rows (W rows above T rows, so one MMA yields O and U together) of NP
    // bf16 columns, each row in a 128-byte line of its own with the 128-byte swizzle (NP < 64 leaves the
    // rest of the line empty), once for the hi parts and once for the lo parts; they overlay the stage's
    // dead [Q;K] tile
    static constexpr int PART = 2 * NP * 128;
    static constexpr int OFF_W_HI = 0, OFF_T_HI = NP * 128;
    static constexpr int OFF_W_LO = PART, OFF_T_LO = OFF_W_LO + NP * 128;
    static constexpr int TILE_BYTES = 2 * PART;
    static_assert(TILE_BYTES <= QK_BYTES, "operand overlays fit");
    // scratch over the dead tiles: the raw Gram rows (up to 32 nodes: in the S0 tile, beside the B
    // tiles; 64 nodes: the stash IS the [Q;K] tile, rows of NP floats with their 16-byte columns swizzled
    // by the row number, and the B tiles, zeroed once the lists are built, take its place), so that with
    // 64 nodes a state tile is dead once stage 1 has read it.  Trees with a path of more than 8
    // ancestors ("deep") need more: their back-substitution rows and full-length lists.  Up to 32 nodes
    // both are in the S0 tile; with 64 nodes a deep tree keeps its S0 tile until stage 2 ends, the lists
    // A and P (NP x NP floats each) fill it exactly, the ancestors' indices take the place of the slot's
    // short lists, and the rows live in the solver threads' local memory.
    static constexpr int RLD = BIG ? NP : NP + 4;  // row stride of the raw Gram stash (floats)
    static constexpr int XLD = NP + 1;
    static constexpr int OFF_RAW = BIG ? 0 : OFF_S0, OFF_XR = OFF_S0 + 2 * NP * RLD * 4;  // (OFF_XR: up to 32 nodes)
    static_assert(OFF_RAW + 2 * NP * RLD * 4 <= (BIG ? QK_BYTES : OFF_S0 + S0_BYTES), "Gram stash fits");
    static constexpr int OFF_DAP = OFF_S0 + (2 * NP * RLD * 4 + 2 * NP * XLD * 4 + 15) / 16 * 16;  // (up to 32 nodes)
    static constexpr int OFF_DPP = OFF_DAP + NP * NP * 4, OFF_DIDX = OFF_DPP + NP * NP * 4;
    static_assert(BIG || OFF_DIDX + NP * NP <= OFF_S0 + S0_BYTES, "scratch fits in the S0 tile");
    static_assert(!BIG || 2 * NP * NP * 4 == S0_BYTES, "64 nodes: the full-length lists fill a state tile");
    static constexpr int V_BYTES = NP * D * 2;
    // a slot (consecutive items alternate between the two): path lists of the first 8 ancestors,
    // per-node scalars, and the item's v rows [NP][128] bf16
    static constexpr int GP_AP = 0, GP_PP = 2 * NP * 16, GP_SCAL = 4 * NP * 16;
    static constexpr int GP_VS = (GP_SCAL + NP * 16 + 127) / 128 * 128;
    static constexpr int GP_BYTES = GP_VS + V_BYTES;
    static_assert(!BIG || GP_SCAL >= NP * NP, "64 nodes: a deep tree's ancestor indices fit over the slot's short lists");
    static constexpr int OFF_S0R = STAGES * STAGE_BYTES;  // (S0_RING) the ring of state tiles
    static constexpr int OFF_GP = OFF_S0R + (S0_RING ? S0_SLOTS * S0_BYTES : 0);
    static constexpr int OFF_MRING = OFF_GP + SLOTS * GP_BYTES;  // 64 nodes: the ring of meta blocks
    static constexpr int OFF_EINFO = OFF_MRING + (META_RING ? META_SLOTS * META_STRIDE : 0);  // (n, first output row) of the item in a TMEM block
    // fused mode: operands of the commit's rank-P product, K-major without swizzle, K = 8 path nodes:
    // core matrices of 8 rows x 16 bytes, the two K halves COPS_LBO apart
    static constexpr int COPS_LBO = D * 16, COPS_TILE = 2 * COPS_LBO;
    static constexpr int OFF_CA_HI = (OFF_EINFO + TBUF * 8 + 127) / 128 * 128;
    static constexpr int OFF_CA_LO = OFF_CA_HI + COPS_TILE, OFF_CB = OFF_CA_LO + COPS_TILE;
    static constexpr int OFF_BAR = FUSED ? OFF_CB + COPS_TILE : OFF_EINFO + TBUF * 8;
    // work list of a launch that takes one size class of a mixed batch: the CTA's units of that class
    // (up to CT_CAP of them; a longer list is walked whole), then 32 warp counts
    static constexpr int CT_CAP = 1024;
    static constexpr int OFF_CTAB = OFF_BAR + (5 * STAGES + 4 * TBUF + RBUF + 5 * SLOTS + 1) * 8 + 16;
    static constexpr int SMEM_BYTES = OFF_CTAB + CT_CAP * 2 + 32 * 4 + 1024;
    static constexpr uint32_t TX_BYTES = S0_BYTES + QK_BYTES;
    // Tensor memory holds two rings.  A block of the first takes SQ | SK from stage 1; the R^T warps
    // turn it, in their own lanes, into g.SQ | 0, stage 2 accumulates [O | U] on top, and the
    // epilogue frees it.  A block of the second (NP columns) takes the Gram block D2 from stage 1; the
    // Gram warps read it out, the R^T warps write R^T over it as bf16 pairs (two nodes per column: the
    // hi parts in the first NP / 2 columns, the lo parts in the rest), stage 2 takes both as its A
    // operand, and its completion frees the block (long before the epilogue runs).
    static constexpr int TM_COLS = 2 * NP;
    static constexpr int TM_DO = 0, TM_DU = NP;
    static constexpr int TM_R0 = TBUF * TM_COLS;  // second ring
    static constexpr int TM_RCOLS = NP;
    static constexpr int TM_RHI = 0, TM_RLO = NP / 2;
    static constexpr int TM_C0 = TM_R0 + RBUF * TM_RCOLS;  // fused mode: the commit's 128 x 128 accumulator
    static_assert(TM_C0 + (FUSED ? D : 0) <= 512, "tensor memory");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
};

// fused mode: what the commit of the previous round needs for one (sequence, head)
struct PathMeta {
    float w[8];               // e^{L_a - L_j} of the staged path nodes
    unsigned long long mask;  // ancestor-or-self mask of the accepted node (previous tree)
    float La, ga;             // its log-gate and e^{La}
    int plen;                 // path length; -1 = no commit for this item
    int lo;                   // first packed node of the sequence in the previous tree
    int h;                    // the item's value head
};
static_assert(sizeof(PathMeta) <= 128, "path meta block");

// (CLASS: the launch takes one size class of a mixed batch and walks a compacted work list; TU: the
// type U is stored in, float or __half.  Both are template parameters because the code they add
// costs the other launches instruction-cache hits: 2 % of the headline kernel's time for either.)
template <int NP, typename TOut, bool FUSED, bool CLASS, typename TU>
__global__ void __launch_bounds__(VtCfg<NP, FUSED>::THREADS, 1)
verify_sm100_tc_kernel(VerifyArgs a, PrevRound pv, int n_items, const __grid_constant__ CUtensorMap tmS0,
                       const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV)
{
    using C = VtCfg<NP, FUSED>;
    // ancestor masks of this round's trees as the kernel handles them: 32 bits (cheaper) up to 32 nodes
    using mask_t = typename std::conditional<(NP > 32), unsigned long long, uint32_t>::type;
    auto m_ffs = [](mask_t m) { return (NP > 32 ? __ffsll((long long)m) : __ffs((int)m)) - 1; };
    auto m_popc = [](mask_t m) { return NP > 32 ? __popcll(m) : __popc((uint32_t)m); };
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint64_t *empty = full + C::STAGES;
    uint64_t *mma1_done = empty + C::STAGES;
    uint64_t *ops_ready = mma1_done + C::TBUF;
    uint64_t *mma2_done = ops_ready + C::TBUF;
    uint64_t *tmem_free = mma2_done + C::TBUF;
    uint64_t *r_free = tmem_free + C::TBUF;
    uint64_t *v_ready = r_free + C::RBUF;              // v rows of a slot have landed
    uint64_t *v_free = v_ready + C::SLOTS;             // R^T warps -> fetching thread: v rows copied to registers
    uint64_t *lists_ready = v_free + C::SLOTS;         // Gram warps -> solver / R^T warps: lists and scalars written
    uint64_t *lists_free = lists_ready + C::SLOTS;     // solver + R^T warps -> Gram warps: the slot may be rewritten
    uint64_t *scal_ready = lists_free + C::SLOTS;      // Gram warps -> R^T warps: per-node scalars written
    uint64_t *upd_done = scal_ready + C::SLOTS;        // fused mode: the state tile of a stage carries the commit
    uint64_t *cmma_done = upd_done + C::STAGES;        // fused mode: the commit's rank-P product has finished
    uint64_t *s0_empty = cmma_done + 1;                // 64 nodes: a tile of the S0 ring may be refilled
    uint64_t *s0_full = s0_empty + C::STAGES;          //           ... has landed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(s0_full + C::STAGES);
    int2 *einfo = reinterpret_cast<int2 *>(smem + C::OFF_EINFO);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Item kk of this CTA (>= n_items when there is none).  When an even number of value heads
    // share a q/k head, a CTA takes the heads two by two: both items of a pair have the same tree
    // and the same [Q;K] rows, so the second reuses the first one's Gram entries.
    const bool pair_mode = ((a.H_v / a.H_qk) & 1) == 0;
    // The CTA's units (items, or pairs of them) are numbers blockIdx.x, blockIdx.x + gridDim.x, ... of the
    // launch's units.  A launch that takes one size class of a mixed batch numbers only the units of the
    // sequences of its class, over the whole batch, so that every CTA gets the same share of them whatever
    // their places in the batch; its own units are then listed in ctab (see the prologue below).  A batch of
    // more than CT_CAP sequences is walked whole.
    const int ups = pair_mode ? a.H_v >> 1 : a.H_v;  // units per sequence
    // (a unit's number has to fit the table's 16 bits, and a CTA's units the table)
    const bool compact = CLASS && a.B <= C::CT_CAP && a.B * ups <= 65536 &&
                         (a.B * ups + (int)gridDim.x - 1) / (int)gridDim.x <= C::CT_CAP;
    int K = 0;  // compact: the CTA's units (set by the prologue)
    const uint16_t *ctab = reinterpret_cast<const uint16_t *>(smem + C::OFF_CTAB);
    auto item_of = [&](int kk) {
        const int ku = pair_mode ? kk >> 1 : kk;
        if constexpr (CLASS) {
            if (compact) {
                if (ku >= K) return n_items;
                const int unit = ctab[ku];  // sequence * ups + unit of the sequence
                return pair_mode ? 2 * unit + (kk & 1) : unit;
            }
        }
        const int g = (int)blockIdx.x + ku * (int)gridDim.x;
        return pair_mode ? 2 * g + (kk & 1) : g;
    };

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int i = 0; i < C::TBUF; ++i) {
            ptx::mbar_init(&mma1_done[i], 2);
            ptx::mbar_init(&ops_ready[i], (C::R_THREADS + C::T_THREADS) / 32);  // one arrival per warp
            ptx::mbar_init(&mma2_done[i], 1);
            ptx::mbar_init(&tmem_free[i], C::E_THREADS / 32);
        }
        for (int i = 0; i < C::RBUF; ++i) ptx::mbar_init(&r_free[i], 1);
        for (int g = 0; g < C::SLOTS; ++g) {
            ptx::mbar_init(&v_ready[g], 1);
            ptx::mbar_init(&v_free[g], C::R_THREADS / 32);
            ptx::mbar_init(&lists_ready[g], C::G_THREADS / 32);
            ptx::mbar_init(&lists_free[g], (C::R_THREADS + C::T_THREADS) / 32);
            ptx::mbar_init(&scal_ready[g], C::G_THREADS / 32);
        }
        for (int s = 0; s < C::STAGES; ++s)
            ptx::mbar_init(&upd_done[s], 128 / 32), ptx::mbar_init(&s0_empty[s], 1), ptx::mbar_init(&s0_full[s], 1);
        ptx::mbar_init(cmma_done, 1);
        ptx::fence_barrier_init();
    }
    if (tid == 32) {  // (the descriptors are kernel parameters: fetched while the kernel before this one still runs)
        ptx::prefetch_tmap(&tmS0), ptx::prefetch_tmap(&tmQ);
        ptx::prefetch_tmap(&tmK), ptx::prefetch_tmap(&tmV);
    }
    if (warp == C::MMA1_WARP) {
        ptx::tmem_alloc(tmem_slot, VT_TMEM_COLS);
        ptx::tmem_relinquish();
        ptx::tc_fence_before_sync();
    }
    grid_dependency_wait();  // the kernel before this one on the stream has finished: global memory may be read
    if (tid == 0) ptx::wait_deadline_init(a.wait_cycles);
    __syncthreads();
    grid_dependency_trigger();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (CLASS && compact) {
        // Every role would otherwise hand every unit of the other classes through the whole pipeline
        // just to drop it (a third of the time of a ragged batch).  First the sequences of the class, over
        // the whole batch: all threads, one sequence each per round, kept sequences numbered by warp
        // ballots and a prefix over the warps' counts (scratch: the first stage, idle until the roles
        // start).  Then this CTA's units, numbers blockIdx.x, blockIdx.x + gridDim.x, ... of the kept
        // sequences' units, into ctab: a role finds its item with one load.
        uint16_t *seq = reinterpret_cast<uint16_t *>(smem);
        uint16_t *tab = reinterpret_cast<uint16_t *>(smem + C::OFF_CTAB);
        int *wcount = reinterpret_cast<int *>(smem + C::OFF_CTAB + C::CT_CAP * 2);
        int kept = 0;
        for (int base = 0; base < a.B; base += C::THREADS) {
            const int b = base + tid;
            bool keep = false;
            if (b < a.B) {
                const int lo = a.node_offsets[b], n = a.node_offsets[b + 1] - lo;
                // another class's well-formed sequence goes; whatever has to be flagged stays
                keep = !(n >= 1 && n <= a.max_nodes && (n <= a.cls_lo || n > a.cls_hi || n > NP)) || bad_offsets(lo, n, a.T) ||
                       (a.cls_lo == 0 && state_slot(a.state_index, a.n_states, b) < 0);
            }
            const uint32_t bal = __ballot_sync(0xffffffffu, keep);
            if (lane == 0) wcount[warp] = __popc(bal);
            __syncthreads();
            int before = 0, total = 0;
#pragma unroll 1
            for (int w2 = 0; w2 < C::THREADS / 32; ++w2) {
                const int c = wcount[w2];
                before += w2 < warp ? c : 0, total += c;
            }
            if (keep) seq[kept + before + __popc(bal & ((1u << lane) - 1u))] = (uint16_t)b;
            kept += total;
            __syncthreads();
        }
        const int n_units = kept * ups;  // (at most 65536: a unit's number fits 16 bits)
        K = n_units > (int)blockIdx.x ? (n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
        for (int ku = tid; ku < K; ku += C::THREADS) {
            const int g = (int)blockIdx.x + ku * (int)gridDim.x, sq = g / ups;
            tab[ku] = (uint16_t)((int)seq[sq] * ups + (g - sq * ups));
        }
        __syncthreads();
    }

    // the state tile of item kk of this CTA
    auto s0_of = [&](int kk) {
        return C::S0_RING ? smem + C::OFF_S0R + (kk % C::S0_SLOTS) * C::S0_BYTES
                          : smem + (kk % C::STAGES) * C::STAGE_BYTES + C::OFF_S0;
    };
    // the meta block of item kk of this CTA
    auto meta_of = [&](int kk) {
        return C::META_RING ? smem + C::OFF_MRING + (kk % C::META_SLOTS) * C::META_STRIDE
                            : smem + (kk % C::STAGES) * C::STAGE_BYTES + C::OFF_META;
    };
    auto meta_mask = [&](unsigned char *mt) { return reinterpret_cast<unsigned long long *>(mt); };
    auto meta_L = [&](unsigned char *mt) { return reinterpret_cast<float *>(mt + NP * 8); };
    auto meta_beta = [&](unsigned char *mt) { return reinterpret_cast<float *>(mt + NP * 12); };
    auto meta_nlo = [&](unsigned char *mt) { return reinterpret_cast<int *>(mt + NP * 16); };
    auto meta_rat = [&](unsigned char *mt) { return reinterpret_cast<float4 *>(mt + C::META_RAT); };
    auto meta_idx = [&](unsigned char *mt) { return reinterpret_cast<uint32_t *>(mt + C::META_IDX); };
    // element (row, col) of the raw Gram stash
    auto raw_at = [](int row, int col) {
        return C::BIG ? row * C::RLD + ((((col >> 2) ^ (row & 15)) << 2) | (col & 3)) : row * C::RLD + col;
    };
    // byte offset of element (row, col) of a stage-2 B tile (bf16, one 128-byte line per row, 128-byte swizzle)
    auto tile_off = [](int row, int col) { return row * 128 + (((col >> 3) ^ (row & 7)) << 4) + ((col & 7) << 1); };

    if (C::S0_RING && warp == C::S0P_WARP) {
        // ------------------------------------------------------------------ state-tile warp (64 nodes)
        // Fills the ring of S0 tiles in item order: a tile's address depends on nothing but the item's
        // number (and the sequence's state slot), so this warp validates nothing; an item the pipeline
        // skips gets its tile all the same (stage 1 waits for it before it hands the slot back).
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            if (item == a.skip_item) continue;  // test hook: this item's loads and their arrival never happen
            const int b = item / a.H_v, h = item - b * a.H_v;
            const int slot = state_slot(a.state_index, a.n_states, b);
            const int srow = (slot < 0 ? 0 : slot) * a.H_v + h;
            const int z = kk % C::S0_SLOTS;
            if (!ptx::mbar_wait(&s0_empty[z], ((kk / C::S0_SLOTS) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], TREEWY_SEQ_TIMEOUT);
                break;
            }
            if (lane == 0) {
                unsigned char *tile = s0_of(kk);
                ptx::mbar_arrive_expect_tx(&s0_full[z], C::S0_BYTES);
                ptx::tma_load_2d(tile, &tmS0, 0, srow * D, &s0_full[z]);
                ptx::tma_load_2d(tile + C::S0_HALF, &tmS0, 64, srow * D, &s0_full[z]);
            }
            __syncwarp();
        }
    } else if (warp >= C::PROD_WARP0) {
        // ------------------------------------------------------------------ producer warp
        const int s = warp - C::PROD_WARP0;
        unsigned char *stage = smem + s * C::STAGE_BYTES;
        const int group = a.H_v / a.H_qk;
        // Node scalars of an item: validated and loaded one round ahead (software pipeline), so the
        // dependent chain  node_offsets -> parent / mask / log-gate / beta  never delays a TMA issue.
        struct Pre {
            int item, b, h, lo, n, bad, flag;
            int srow;  // state tile of the item: (state slot) * H_v + h
            unsigned long long mk[C::NPL];  // lane l owns nodes l, l + 32
            float Lv[C::NPL], bv[C::NPL];
            int deep;  // whether any path has more than 8 ancestors
            // fused mode: the previous round's accepted path of this sequence
            int plo, pbad, plen, cnt, pj;
            unsigned long long pmask;
            float La, wj;
        };
        auto fetch = [&](int kk) {
            Pre p;
            p.item = item_of(kk);
            p.b = 0, p.h = 0, p.lo = 0, p.n = 0, p.bad = 0, p.flag = 1, p.srow = 0;
#pragma unroll
            for (int r = 0; r < C::NPL; ++r) p.mk[r] = 0ull, p.Lv[r] = 0.f, p.bv[r] = 0.f;
            p.deep = 0;
            p.plo = 0, p.pbad = 0, p.plen = -1, p.cnt = 0, p.pj = 0, p.pmask = 0ull, p.La = 0.f, p.wj = 0.f;
            if (p.item >= n_items) return p;
            p.b = p.item / a.H_v, p.h = p.item - p.b * a.H_v;
            p.lo = a.node_offsets[p.b];
            p.n = a.node_offsets[p.b + 1] - p.lo;
            const int slot = state_slot(a.state_index, a.n_states, p.b);
            p.srow = (slot < 0 ? 0 : slot) * a.H_v + p.h;
            if (slot < 0) {
                p.bad = TREEWY_SEQ_BAD_STATE;
                p.flag = a.cls_lo == 0;
            } else if (bad_offsets(p.lo, p.n, a.T)) {
                p.bad = TREEWY_SEQ_BAD_OFFSETS;
                p.flag = a.cls_lo == 0;
            } else if (p.n < 1 || p.n > a.max_nodes) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES;
                p.flag = a.cls_lo == 0;
            } else if (p.n <= a.cls_lo || p.n > a.cls_hi || p.n > NP) {
                p.bad = TREEWY_SEQ_TOO_MANY_NODES;  // another launch's size class: skipped, not flagged
                p.flag = 0;
            } else {
                bool bp = false;
#pragma unroll
                for (int r = 0; r < C::NPL; ++r) {
                    const int i = lane + 32 * r;
                    const int par = i < p.n ? a.parent[p.lo + i] : -1;
                    bp |= i < p.n && (par < -1 || par >= i);
                }
                if (__any_sync(0xffffffffu, bp)) p.bad = TREEWY_SEQ_BAD_PARENT;
            }
            bool dp8 = false;
#pragma unroll
            for (int r = 0; r < C::NPL; ++r) {
                const int i = lane + 32 * r;
                const bool on = !p.bad && i < p.n;
                p.mk[r] = on ? a.anc_mask[p.lo + i] : 0ull;
                p.Lv[r] = on ? a.cum_log_gate[(size_t)(p.lo + i) * a.H_v + p.h] : 0.f;
                p.bv[r] = on ? a.beta[(size_t)(p.lo + i) * a.H_v + p.h] : 0.f;
                dp8 |= m_popc((mask_t)p.mk[r] & ~((mask_t)1 << i)) > 8;
            }
            p.deep = __any_sync(0xffffffffu, dp8);
            if constexpr (FUSED) {
                p.plo = pv.node_offsets[p.b];
                const int pn = pv.node_offsets[p.b + 1] - p.plo;
                const int acc = pv.accepted[p.b];
                if (slot < 0) {
                    p.pbad = TREEWY_SEQ_BAD_STATE;  // no state to commit into
                } else if (bad_offsets(p.plo, pn, pv.T)) {
                    p.pbad = TREEWY_SEQ_BAD_OFFSETS;
                } else if (pn < 1 || pn > pv.max_nodes) {
                    p.pbad = TREEWY_SEQ_TOO_MANY_NODES;
                } else {
                    int bp = 0;
#pragma unroll 1
                    for (int i = lane; i < pn; i += 32) {
                        const int par = pv.parent[p.plo + i];
                        bp |= (par < -1 || par >= i);
                    }
                    if (__any_sync(0xffffffffu, bp)) p.pbad = TREEWY_SEQ_BAD_PARENT;
                    else if (acc < -1 || acc >= pn) p.pbad = TREEWY_SEQ_BAD_ACCEPTED;
                }
                if (!p.pbad && acc >= 0) {
                    p.pmask = pv.anc_mask[p.plo + acc];
                    p.La = pv.cum_log_gate[(size_t)(p.plo + acc) * a.H_v + p.h];
                    p.plen = __popcll(p.pmask);
                    p.cnt = min(p.plen, C::PCH);
                    if (lane < p.cnt) {
                        p.pj = nth_set_bit(p.pmask, lane);
                        p.wj = __expf(p.La - pv.cum_log_gate[(size_t)(p.plo + p.pj) * a.H_v + p.h]);
                    }
                }
            }
            return p;
        };
        // The first item of a stage: its state tile depends on nothing but the item's number, so it is put
        // in flight before the item's scalars are fetched (two dependent loads, 2 us in a role trace, that
        // would otherwise stand in front of the launch's first bytes).
        const int item0 = item_of(s);
        const bool early = !C::S0_RING && !a.state_index && item0 < n_items && item0 != a.skip_item;
        if (early && lane == 0) {
            uint64_t *bar0 = FUSED ? &s0_full[s] : &full[s];
            ptx::mbar_expect_tx(bar0, C::S0_BYTES);
            ptx::tma_load_2d(stage + C::OFF_S0, &tmS0, 0, item0 * D, bar0);
            ptx::tma_load_2d(stage + C::OFF_S0 + C::S0_HALF, &tmS0, 64, item0 * D, bar0);
        }  // (the q / k rows as well, one load away, was tried: the step got 0.2 % slower, workload 3 1 %)
        // An item's meta block: node scalars, size and place, and the path lists of the node(s) a lane owns
        // (index and gate ratio e^{L_i - L_j} of the first 8 ancestors; only the ratios depend on the head).
        // Building the lists here takes the ffs / exp chain off the consumers' critical path.  (Rolled:
        // code size.  Building them in registers, the other nodes' log-gates by shuffle, was tried: the
        // unrolled code made every instance slower, 2 % to 5 %.)
        auto write_meta = [&](const Pre &p, unsigned char *mt) {
#pragma unroll
            for (int r = 0; r < C::NPL; ++r) {
                const int i = lane + 32 * r;
                if (i < NP) meta_mask(mt)[i] = p.mk[r], meta_L(mt)[i] = p.Lv[r], meta_beta(mt)[i] = p.bv[r];
            }
            if (lane == 0)
                meta_nlo(mt)[0] = p.bad ? 0 : p.n, meta_nlo(mt)[1] = p.lo * a.H_v + p.h, meta_nlo(mt)[2] = p.deep,
                meta_nlo(mt)[3] = p.srow;
            __syncwarp();  // the log-gates of all nodes are in the meta block
            const float *Lm = meta_L(mt);
#pragma unroll
            for (int r = 0; r < C::NPL; ++r) {
                const int i = lane + 32 * r;
                mask_t m = (mask_t)p.mk[r] & ~((mask_t)1 << i);
                float *ratp = reinterpret_cast<float *>(meta_rat(mt)) + i * 4;
                unsigned char *idxp = reinterpret_cast<unsigned char *>(meta_idx(mt)) + i * 4;
#pragma unroll 1
                for (int d = 0; d < 8; ++d) {
                    const int j = m ? m_ffs(m) : 0;
                    const float rt = m ? __expf(p.Lv[r] - Lm[j]) : 0.f;
                    if (i < NP) ratp[(d >> 2) * NP * 4 + (d & 3)] = rt, idxp[(d >> 2) * NP * 4 + (d & 3)] = (unsigned char)j;
                    m &= m - 1;
                }
            }
        };
        // (One call site for the fetch: it is the largest piece of code a producer runs.  The loop's first
        // round, kk = s - STAGES, only fetches; a round processes the item fetched by the round before.)
        Pre cur = {};
        bool s0_issued = early;  // the state tile of `cur` is in flight already
#pragma unroll 1
        for (int kk = s - C::STAGES;; kk += C::STAGES) {
            // (test hook: the skipped item's loads and their arrival never happen)
            if (kk >= s && cur.item >= n_items) break;
            if (kk >= s && cur.item != a.skip_item) {
            const Pre p = cur;
            unsigned char *mt = meta_of(kk);
            if constexpr (C::META_RING) write_meta(p, mt);  // the block of item kk - 2 * STAGES: long read
            if (p.bad && p.flag && p.h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], p.bad);
            if (FUSED && p.pbad && p.h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], p.pbad);
            if (!ptx::mbar_wait(&empty[s], ((kk / C::STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[p.b], TREEWY_SEQ_TIMEOUT);
                break;
            }
            if constexpr (FUSED) {
                PathMeta *pm = reinterpret_cast<PathMeta *>(stage + C::OFF_PMETA);
                if (lane < p.cnt) pm->w[lane] = p.wj;
                if (lane == 0) pm->mask = p.pmask, pm->La = p.La, pm->ga = __expf(p.La), pm->plen = p.plen, pm->lo = p.plo, pm->h = p.h;
            }
            // The copies are issued first and announced (expect_tx, with the warp's one arrival) last:
            // the phase cannot complete before that arrival, and the path lists below are written
            // while the data is on its way.
            const bool tile_issued = s0_issued;
            // the state tile serves verify, commit or both (64 nodes: it comes through the ring of its own)
            const bool need_tile = !C::S0_RING && (!p.bad || p.plen >= 0) && !tile_issued;
            // Fused mode: what the commit group waits for (state tile, the previous round's path rows, the
            // path meta block) is announced on a barrier of its own, as soon as it has been issued: the
            // group starts when THAT has landed, not when the last of the q / k rows has (the copies of a
            // stage are accepted one after the other, ~200 cycles each).
            uint64_t *cbar = FUSED ? &s0_full[s] : &full[s];
            const uint32_t tx_c = (need_tile ? C::S0_BYTES : 0) + p.cnt * (D * 2 + D * 4);
            const uint32_t tx_q = p.bad ? 0 : C::QK_BYTES;
            const uint32_t tx = FUSED ? tx_q : tx_c + tx_q;
            const int hq = p.h / group;
            if (lane == 0 && need_tile) {
                ptx::tma_load_2d(stage + C::OFF_S0, &tmS0, 0, p.srow * D, cbar);
                ptx::tma_load_2d(stage + C::OFF_S0 + C::S0_HALF, &tmS0, 64, p.srow * D, cbar);
            }
            if constexpr (FUSED) {
                __syncwarp();
                if (lane < p.cnt) {  // the accepted path's k and U rows of the previous round
                    const __nv_bfloat16 *kp = static_cast<const __nv_bfloat16 *>(pv.k);
                    ptx::bulk_g2s(stage + C::OFF_KP + lane * D * 2,
                                  kp + ((size_t)(p.plo + p.pj) * a.H_qk + hq) * D, D * 2, cbar);
                    ptx::bulk_g2s(stage + C::OFF_UP + lane * D * 4, pv.U + ((size_t)(p.plo + p.pj) * a.H_v + p.h) * D,
                                  D * 4, cbar);
                }
                __syncwarp();
                if (lane == 0) {
                    if (tx_c == 0) ptx::mbar_arrive(cbar);
                    else ptx::mbar_arrive_expect_tx(cbar, tx_c);
                }
            }
            if (lane == 0 && !p.bad) {
                ptx::tma_load_2d(stage, &tmQ, hq * D, p.lo, &full[s]);
                ptx::tma_load_2d(stage + C::QK_HALF, &tmQ, hq * D + 64, p.lo, &full[s]);
                ptx::tma_load_2d(stage + NP * 128, &tmK, hq * D, p.lo, &full[s]);
                ptx::tma_load_2d(stage + C::QK_HALF + NP * 128, &tmK, hq * D + 64, p.lo, &full[s]);
            }
            if constexpr (!C::META_RING) write_meta(p, mt);  // (while the data is on its way)
            __syncwarp();
            if (lane == 0) {
                if (tx == 0) ptx::mbar_arrive(&full[s]);
                else ptx::mbar_arrive_expect_tx(&full[s], tx);
            }
            }
            cur = fetch(kk + C::STAGES);  // in flight while this stage is being consumed
            if (kk >= s) s0_issued = false;
        }
    } else if (FUSED && warp >= C::COMMIT_WARP0 && warp < C::MMA1_WARP) {
        // ------------------------------------------------------------------ commit group (fused mode)
        // Before the stage-1 MMAs read a state tile, the previous round's accepted node is
        // committed INTO it (Eq. 3):  S <- g_a S + sum_{j on the path} (g_a / g_j) u_j k_j^T .
        // The rank-P term is a tensor-core product, 8 path nodes per round:
        //   C[v][c] (+)= sum_p A[v][p] B[c][p],  A[v][p] = (g_a / g_p) u_p[v] (fp32 as tf32 hi + lo),
        //   B[c][p] = k_p[c] (bf16, exact in tf32),
        // both operands written by this group, K-major without swizzle; thread t owns row t of A, row
        // t of B and, afterwards, TMEM lane t = row t of the state.  Then S[t][:] = g_a S[t][:] + C[t][:]
        // is rounded once to bf16 in place (the tile keeps the 128-byte swizzle the TMA gave it), and
        // the new state goes back to global memory with a TMA store while verification proceeds from
        // the shared-memory copy.
        const int t = tid - C::COMMIT_WARP0 * 32;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tC = tmem_base + lane_base + C::TM_C0;
        const int group = a.H_v / a.H_qk;
        constexpr uint32_t idescC = ptx::umma_idesc_tf32_f32(128, D);
        unsigned char *opA_hi = smem + C::OFF_CA_HI, *opA_lo = smem + C::OFF_CA_LO, *opB = smem + C::OFF_CB;
        const int op_off = (t >> 3) * 128 + (t & 7) * 16;  // this thread's row in a core-matrix column
        uint32_t rounds = 0;  // completed rank-P products: parity of cmma_done
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            if (!ptx::mbar_wait(&s0_full[s], (kk / C::STAGES) & 1)) {  // state tile, path rows, path meta
                if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            const PathMeta *pm = reinterpret_cast<const PathMeta *>(stage + C::OFF_PMETA);
            const int plen = pm->plen;
            if (plen >= 0) {
                const int h = pm->h;
                const __nv_bfloat16 *kp = reinterpret_cast<const __nv_bfloat16 *>(stage + C::OFF_KP);
                const float *up = reinterpret_cast<const float *>(stage + C::OFF_UP);
                const __nv_bfloat16 *kg = static_cast<const __nv_bfloat16 *>(pv.k);
                unsigned long long m = pm->mask;  // path nodes not yet taken (rounds beyond the staged rows)
                bool ok = true;
#pragma unroll 1
                for (int r0 = 0; r0 < plen && ok; r0 += 8) {
                    if (r0 == 0) {  // the rows the producer staged (C::PCH = 8)
                        float av[8], bv[8];
#pragma unroll
                        for (int p = 0; p < 8; ++p) {
                            const float u = up[p * D + t], kf = __bfloat162float(kp[p * D + t]);
                            av[p] = p < plen ? pm->w[p] * u : 0.f;  // rows past the path hold stale data
                            bv[p] = p < plen ? kf : 0.f;
                        }
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            float4 hi, lo;
                            hi.x = ptx::tf32_hi(av[4 * c]), hi.y = ptx::tf32_hi(av[4 * c + 1]);
                            hi.z = ptx::tf32_hi(av[4 * c + 2]), hi.w = ptx::tf32_hi(av[4 * c + 3]);
                            lo.x = av[4 * c] - hi.x, lo.y = av[4 * c + 1] - hi.y;
                            lo.z = av[4 * c + 2] - hi.z, lo.w = av[4 * c + 3] - hi.w;
                            *reinterpret_cast<float4 *>(opA_hi + c * C::COPS_LBO + op_off) = hi;
                            *reinterpret_cast<float4 *>(opA_lo + c * C::COPS_LBO + op_off) = lo;
                            *reinterpret_cast<float4 *>(opB + c * C::COPS_LBO + op_off) =
                                make_float4(bv[4 * c], bv[4 * c + 1], bv[4 * c + 2], bv[4 * c + 3]);
                        }
#pragma unroll 1
                        for (int p = 0; p < 8; ++p) m &= m - 1;
                    } else {  // deep path: straight from global memory, one node at a time (rolled: code size)
#pragma unroll 1
                        for (int p = 0; p < 8; ++p) {
                            float av = 0.f, bv = 0.f;
                            if (r0 + p < plen) {
                                const int j = __ffsll((long long)m) - 1;
                                const float w = __expf(pm->La - pv.cum_log_gate[(size_t)(pm->lo + j) * a.H_v + h]);
                                av = w * pv.U[((size_t)(pm->lo + j) * a.H_v + h) * D + t];
                                bv = __bfloat162float(kg[((size_t)(pm->lo + j) * a.H_qk + h / group) * D + t]);
                            }
                            m &= m - 1;
                            const int off = (p >> 2) * C::COPS_LBO + op_off + (p & 3) * 4;
                            const float hi = ptx::tf32_hi(av);
                            *reinterpret_cast<float *>(opA_hi + off) = hi;
                            *reinterpret_cast<float *>(opA_lo + off) = av - hi;
                            *reinterpret_cast<float *>(opB + off) = bv;
                        }
                    }
                    ptx::fence_proxy_async();  // operands were written by ordinary stores
                    ptx::tc_fence_before_sync();
                    ptx::named_sync(3, C::CGROUP > 0 ? C::CGROUP : 32);
                    if (t == 0) {
                        ptx::tc_fence_after_sync();
                        const uint64_t dB = ptx::umma_desc_k_plain(ptx::smem_u32(opB), C::COPS_LBO, 128);
                        ptx::umma_tf32(tmem_base + C::TM_C0, ptx::umma_desc_k_plain(ptx::smem_u32(opA_hi), C::COPS_LBO, 128),
                                       dB, idescC, r0 > 0);
                        ptx::umma_tf32(tmem_base + C::TM_C0, ptx::umma_desc_k_plain(ptx::smem_u32(opA_lo), C::COPS_LBO, 128),
                                       dB, idescC, 1u);
                        ptx::umma_commit(cmma_done);
                    }
                    ok = ptx::mbar_wait(cmma_done, rounds & 1);
                    ++rounds;
                    ptx::tc_fence_after_sync();
                }
                if (!ok) {  // the product never finished: the tile keeps the old state, nothing is stored
                    if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                    break;
                }
                // S[t][:] = g_a S[t][:] + C[t][:], sixteen columns at a time; the next sixteen columns of
                // C are on their way from tensor memory while the current ones are worked on
                const float ga = pm->ga;
                unsigned char *row = stage + C::OFF_S0 + t * 128;
                auto fix16 = [&](int c0, const uint32_t (&d)[16]) {
                    unsigned char *half = row + (c0 >> 6) * C::S0_HALF;
                    const int ch = (c0 & 63) >> 3;  // 16-byte chunk inside the 128-byte row
                    uint4 *p0 = reinterpret_cast<uint4 *>(half + (((ch) ^ (t & 7)) << 4));
                    uint4 *p1 = reinterpret_cast<uint4 *>(half + (((ch + 1) ^ (t & 7)) << 4));
                    float s0[8], s1[8];
                    widen8(*p0, s0);
                    widen8(*p1, s1);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        s0[e] = fmaf(ga, s0[e], __uint_as_float(d[e]));
                        s1[e] = fmaf(ga, s1[e], __uint_as_float(d[8 + e]));
                    }
                    uint4 y0, y1;
                    y0.x = pack_bf16(s0[0], s0[1]), y0.y = pack_bf16(s0[2], s0[3]);
                    y0.z = pack_bf16(s0[4], s0[5]), y0.w = pack_bf16(s0[6], s0[7]);
                    y1.x = pack_bf16(s1[0], s1[1]), y1.y = pack_bf16(s1[2], s1[3]);
                    y1.z = pack_bf16(s1[4], s1[5]), y1.w = pack_bf16(s1[6], s1[7]);
                    *p0 = y0, *p1 = y1;
                };
                uint32_t da[16], db[16];
                ptx::tmem_ld16(tC, da);
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 32) {
                    ptx::tmem_wait_ld();
                    ptx::tmem_ld16(tC + c0 + 16, db);
                    fix16(c0, da);
                    ptx::tmem_wait_ld();
                    if (c0 + 32 < D) ptx::tmem_ld16(tC + c0 + 32, da);
                    fix16(c0 + 16, db);
                }
                ptx::tc_fence_before_sync();
                ptx::fence_proxy_async();  // the tile is read next by the tensor core and by the TMA store
            }
            ptx::mbar_arrive_warp(&upd_done[s]);  // (the first stage-1 MMA warp sends the new state to global memory)
        }
    } else if (warp == C::MMA1_WARP || warp == C::MMA1B_WARP) {
        // ------------------------------------------------------------------ stage-1 MMAs
        // One tcgen05.mma of these sizes keeps its issuing thread for ~120 cycles, so the two
        // accumulation chains (S0 [Q;K]^T and the Gram block) are issued by two warps.
        const bool gram_chain = warp == C::MMA1B_WARP;
        constexpr uint32_t idesc1 = ptx::umma_idesc_bf16_f32(128, 2 * NP);
        constexpr uint32_t idesc2 = ptx::umma_idesc_bf16_f32(128, NP);
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            if (!ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1)) break;
            const bool reuse_gram = pair_mode && (kk & 1) && meta_nlo(mt)[2] == 0;
            const int n = gram_chain && reuse_gram ? 0 : meta_nlo(mt)[0];
            if (FUSED && !ptx::mbar_wait(&upd_done[s], (kk / C::STAGES) & 1)) break;  // tile carries the commit
            bool stored = false;
            if constexpr (FUSED) {
                // the new state goes back to global memory while verification proceeds from this copy.  The
                // Gram chain's warp issues the store (its chain is the shorter one, and idle for the second
                // head of a pair), in front of its MMAs: behind them, the wait for the store to have read the
                // tile delays stage 1's completion signal, 2 % of the launch.
                if (gram_chain && lane == 0 && reinterpret_cast<const PathMeta *>(stage + C::OFF_PMETA)->plen >= 0) {
                    const int srow = meta_nlo(mt)[3];
                    ptx::tma_store_2d(&tmS0, 0, srow * D, stage + C::OFF_S0);
                    ptx::tma_store_2d(&tmS0, 64, srow * D, stage + C::OFF_S0 + C::S0_HALF);
                    ptx::bulk_commit_group();
                    stored = true;
                }
            }
            if (gram_chain) {
                if (!ptx::mbar_wait(&r_free[kk % C::RBUF], ((kk / C::RBUF) & 1) ^ 1)) break;
            } else {
                if (!ptx::mbar_wait(&tmem_free[buf], ((kk / C::TBUF) & 1) ^ 1)) break;
                // (64 nodes: the item's state tile has landed -- also when the item is skipped: the slot
                // goes back below, and its copy must be over by then)
                if (C::S0_RING && !ptx::mbar_wait(&s0_full[kk % C::S0_SLOTS], (kk / C::S0_SLOTS) & 1)) break;
            }
            ptx::tc_fence_after_sync();
            if (lane == 0) {
                if (n > 0) {
                    const uint32_t qk = ptx::smem_u32(stage), s0 = ptx::smem_u32(s0_of(kk));
                    const uint32_t d1 = tmem_base + buf * C::TM_COLS;
                    const uint32_t d2 = tmem_base + C::TM_R0 + (kk % C::RBUF) * C::TM_RCOLS;
#pragma unroll 1
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t ko = (ks >> 2) * C::QK_HALF + (ks & 3) * 32;
                        const uint64_t dq = ptx::umma_desc_k_sw128(qk + ko);
                        if (gram_chain) {
                            ptx::umma_bf16(d2, dq, ptx::umma_desc_k_sw128(qk + ko + NP * 128), idesc2, ks > 0);
                        } else {
                            const uint64_t da = ptx::umma_desc_k_sw128(s0 + (ks >> 2) * C::S0_HALF + (ks & 3) * 32);
                            ptx::umma_bf16(d1, da, dq, idesc1, ks > 0);
                        }
                    }
                    // (the Gram warps may write their stash over the state tile once stage 1 is done: the
                    // store must have read it by then)
                    if (stored) ptx::bulk_wait_group_read<0>();
                    ptx::umma_commit(&mma1_done[buf]);
                    if (C::S0_RING && !gram_chain && meta_nlo(mt)[2] == 0) ptx::umma_commit(&s0_empty[kk % C::S0_SLOTS]);
                } else {
                    if (stored) ptx::bulk_wait_group_read<0>();
                    ptx::mbar_arrive(&mma1_done[buf]);
                    if (C::S0_RING && !gram_chain && meta_nlo(mt)[2] == 0) ptx::mbar_arrive(&s0_empty[kk % C::S0_SLOTS]);
                }
            }
            __syncwarp();
        }
        if (FUSED && !gram_chain && lane == 0) ptx::bulk_wait_group<0>();
    } else if (warp == C::MMA2_WARP) {
        // ------------------------------------------------------------------ stage-2 MMAs
        constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(128, 2 * NP);
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            if (!ptx::mbar_wait(&ops_ready[buf], (kk / C::TBUF) & 1)) break;
            ptx::tc_fence_after_sync();
            const int n = meta_nlo(mt)[0];
            const bool keeps_s0 = C::S0_RING && meta_nlo(mt)[2] != 0;  // a deep tree: its S0 tile goes back only now
            if (lane == 0) {
                if (n > 0) {
                    const uint32_t base = ptx::smem_u32(stage);
                    const uint32_t tb = tmem_base + buf * C::TM_COLS;
                    const uint32_t tr = tmem_base + C::TM_R0 + (kk % C::RBUF) * C::TM_RCOLS;
                    // three passes (hi.hi, lo.hi, hi.lo), each NP / 16 steps of K = 16, on top of g.S0q (O)
                    // and zeros (U); rolled: the issue loop is short and code size matters
                    constexpr int KS = NP / 16;
#pragma unroll 1
                    for (int q = 0; q < 3 * KS; ++q) {
                        const int p = q / KS, ks = q % KS;
                        const uint32_t ra = tr + (p == 1 ? C::TM_RLO : C::TM_RHI) + ks * 8;
                        const uint32_t wt = base + (p == 2 ? C::OFF_W_LO : C::OFF_W_HI) + ks * 32;
                        ptx::umma_bf16_ts(tb, ra, ptx::umma_desc_k_sw128(wt), idesc, 1u);
                    }
                    ptx::umma_commit(&mma2_done[buf]);
                    ptx::umma_commit(&empty[s]);  // the stage's operand overlays have been consumed
                    if (keeps_s0) ptx::umma_commit(&s0_empty[kk % C::S0_SLOTS]);
                    ptx::umma_commit(&r_free[kk % C::RBUF]);
                } else {
                    ptx::mbar_arrive(&mma2_done[buf]);
                    ptx::mbar_arrive(&empty[s]);
                    if (keeps_s0) ptx::mbar_arrive(&s0_empty[kk % C::S0_SLOTS]);
                    ptx::mbar_arrive(&r_free[kk % C::RBUF]);
                }
            }
            __syncwarp();
        }
    } else if (warp >= C::G_WARP0 && warp < C::T_WARP0) {
        // ------------------------------------------------------------------ Gram warps
        // Per item: the Gram rows leave tensor memory into a stash, the stage-2 B tiles are zeroed,
        // and the scaled ancestor lists are built for the solver warps:
        //   P[i][d] = e^{L_i-L_j} q_i.k_j ,  A[i][d] = beta_i e^{L_i-L_j} k_i.k_j ,  idx[i][d] = j
        // for j the d-th ancestor of i; lists are stored [d / 4][node][d % 4].
        const int tg = tid - C::G_WARP0 * 32;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const bool gram_reader = (warp - C::G_WARP0) * 32 < 2 * NP;  // warps whose lanes hold [Q;K] rows
        const int i = tg & (NP - 1), kind = (tg / NP) & 1;  // kind 0: P list (q rows), 1: A list (k rows)
        float4 gram4[2];         // this thread's Gram entries (its node's first 8 ancestors), kept for the
        float gram_diag = 0.f;   // second item of a pair; q_i.k_i
        gram4[0] = gram4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF, rb = kk % C::RBUF, L = kk & 1;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            unsigned char *gp = smem + C::OFF_GP + L * C::GP_BYTES;
            float4 *Ap4 = reinterpret_cast<float4 *>(gp + C::GP_AP);
            float4 *Pp4 = reinterpret_cast<float4 *>(gp + C::GP_PP);
            float4 *scal = reinterpret_cast<float4 *>(gp + C::GP_SCAL);
            if (!ptx::mbar_wait(&mma1_done[buf], (kk / C::TBUF) & 1)) {
                if (tg == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            ptx::tc_fence_after_sync();
            ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1);  // already complete: acquires the meta block
            const int n = meta_nlo(mt)[0];
            if (tg == 0) einfo[buf] = make_int2(n, meta_nlo(mt)[1]);
            if (n > 0) {
                const float *Lm = meta_L(mt);
                float *raw = reinterpret_cast<float *>(stage + C::OFF_RAW);
                const bool deep = meta_nlo(mt)[2] != 0;  // some path of this tree has more than 8 ancestors
                // second item of a pair: same tree, same [Q;K] rows; the Gram entries are in registers
                const bool reuse_gram = pair_mode && (kk & 1) && !deep;
                // zero the stage-2 B tiles (they overlay the dead [Q;K] tile; with 64 nodes they also cover
                // the Gram stash and are zeroed further down, once the lists are built)
                if constexpr (!C::BIG) {
                    for (int q = tg; q < C::TILE_BYTES / 16; q += C::G_THREADS)
                        reinterpret_cast<uint4 *>(stage)[q] = make_uint4(0u, 0u, 0u, 0u);
                }
                // the slot's previous lists and scalars must have been read
                if (!ptx::mbar_wait(&lists_free[L], ((kk >> 1) & 1) ^ 1)) break;  // (a role has given up)
                // the rows of the Gram block (row owner = lane)
                if (gram_reader && !reuse_gram) {
                    const uint32_t tr = tmem_base + lane_base + C::TM_R0 + rb * C::TM_RCOLS;
                    constexpr int CH = NP < 32 ? NP : 32;  // columns per read: few, wide reads (each costs a round trip)
#pragma unroll
                    for (int c0 = 0; c0 < NP; c0 += CH) {
                        if (c0 < n) {
                            uint32_t g[CH];
                            if constexpr (CH == 32) ptx::tmem_ld32(tr + c0, g);
                            else ptx::tmem_ld16(tr + c0, g);
                            ptx::tmem_wait_ld();
                            if (tg < 2 * NP) {
#pragma unroll
                                for (int q = 0; q < CH / 4; ++q)
                                    *reinterpret_cast<float4 *>(raw + raw_at(tg, c0 + 4 * q)) = make_float4(__uint_as_float(g[4 * q]), __uint_as_float(g[4 * q + 1]),
                                                         __uint_as_float(g[4 * q + 2]), __uint_as_float(g[4 * q + 3]));
                            }
                        }
                    }
                    ptx::tc_fence_before_sync();
                }
                const bool valid = i < n;
                const float Li = Lm[i];
                const float bi = meta_beta(mt)[i];
                const float scale = kind ? bi : 1.f;
                const int rrow = kind ? NP + i : i;
                // the per-node scalars first (a thread needs only its own row's diagonal entry for them): the
                // R^T warps need nothing else from here, and a warp's arrival says its rows have left tensor memory
                if (tg < NP && valid) {
                    const float gi = __expf(Li);
                    if (!reuse_gram) gram_diag = raw[raw_at(i, i)];
                    scal[i] = make_float4(bi, bi * gi, gi, gram_diag);
                }
                ptx::mbar_arrive_warp(&scal_ready[L]);
                if (!reuse_gram) ptx::named_sync(1, C::G_THREADS);
                if (!deep) {
                    // the producer left indices and gate ratios of the first 8 ancestors: four Gram
                    // entries are scaled at a time, no dependent chain
                    constexpr int HSTEP = C::G_THREADS / (2 * NP), HN = 2 / HSTEP;
#pragma unroll
                    for (int q = 0; q < HN; ++q) {
                        const int hf = tg / (2 * NP) + q * HSTEP;
                        const float4 rt = meta_rat(mt)[hf * NP + i];
                        if (!reuse_gram) {
                            const uint32_t iw = meta_idx(mt)[hf * NP + i];
                            gram4[q] = make_float4(raw[raw_at(rrow, iw & 255u)], raw[raw_at(rrow, (iw >> 8) & 255u)],
                                                   raw[raw_at(rrow, (iw >> 16) & 255u)], raw[raw_at(rrow, iw >> 24)]);
                        }
                        float4 val;
                        val.x = scale * rt.x * gram4[q].x, val.y = scale * rt.y * gram4[q].y;
                        val.z = scale * rt.z * gram4[q].z, val.w = scale * rt.w * gram4[q].w;
                        (kind ? Ap4 : Pp4)[hf * NP + i] = val;
                    }
                } else if (tg < 2 * NP) {
                    // full-length lists, in scratch memory (64 nodes: A and P fill the item's state tile, which
                    // a deep tree keeps until stage 2 ends; the indices take the place of the slot's short lists)
                    unsigned char *dl = C::BIG ? s0_of(kk) : stage + C::OFF_DAP;
                    float *Ap = reinterpret_cast<float *>(dl);
                    float *Pp = reinterpret_cast<float *>(dl + NP * NP * 4);
                    unsigned char *idx = C::BIG ? gp + C::GP_AP : dl + 2 * NP * NP * 4;
                    mask_t m = valid ? (mask_t)meta_mask(mt)[i] & ~((mask_t)1 << i) : (mask_t)0;
#pragma unroll 1
                    for (int d = 0; m; ++d) {
                        const int j = m_ffs(m);
                        m &= m - 1;
                        const float val = scale * __expf(Li - Lm[j]) * raw[raw_at(rrow, j)];
                        const int at = ((d >> 2) * NP + i) * 4 + (d & 3);
                        if (kind) Ap[at] = val;
                        else Pp[at] = val, idx[at] = (unsigned char)j;
                    }
                }
                if constexpr (C::BIG) {  // the stash is dead: the B tiles take its place
                    ptx::named_sync(1, C::G_THREADS);
                    for (int q = tg; q < C::TILE_BYTES / 16; q += C::G_THREADS)
                        reinterpret_cast<uint4 *>(stage)[q] = make_uint4(0u, 0u, 0u, 0u);
                }
                ptx::fence_proxy_async();  // the zero fill is read by the tensor core
            } else {
                if (!ptx::mbar_wait(&lists_free[L], ((kk >> 1) & 1) ^ 1)) break;
                ptx::mbar_arrive_warp(&scal_ready[L]);
            }
            ptx::mbar_arrive_warp(&lists_ready[L]);  // lists and the zero fill are in place
        }
    } else if (warp >= C::T_WARP0 && warp < C::R_WARP0) {
        // ------------------------------------------------------------------ solver warps
        // Rows of T = (I + A)^-1 (one thread per node) and of W = P T (another) by back-substitution
        // along node i's root path j_0 .. j_{dp-1}, j_dp = i:
        //   x_dp = 1 (T) or P[i][i] (W);  x_e = p_e - sum_{f > e} x_f A[j_f][j_e]
        // scattered as bf16 (hi, lo) into the swizzled B tiles of stage 2.  Shared memory only.
        const int tt = tid - C::T_WARP0 * 32;
        const int i = tt & (NP - 1);
        const bool wrow = (tt / NP) & 1;
        // The last solver thread also keeps the v rows coming: as soon as the R^T warps have copied
        // the rows of item k to registers, the slot takes the rows of item k + 2.  Rows past a tree's
        // end belong to other sequences or are zero fill: they are loaded and never used.
        const bool v_thread = tt == C::T_THREADS - 1;
        int v_pending[2] = {-1, -1};  // per slot: the item whose v rows are in flight or unread
        auto first_node = [&](int kx) {
            const int it = item_of(kx);
            return it < n_items ? a.node_offsets[it / a.H_v] : 0;
        };
        auto fetch_v = [&](int kx, int lo_x) {
            const int it = item_of(kx);
            v_pending[kx & 1] = -1;
            if (it >= n_items) return;
            v_pending[kx & 1] = kx;
            ptx::mbar_arrive_expect_tx(&v_ready[kx & 1], C::V_BYTES);
            ptx::tma_load_2d(smem + C::OFF_GP + (kx & 1) * C::GP_BYTES + C::GP_VS, &tmV, (it % a.H_v) * D, lo_x,
                             &v_ready[kx & 1]);
        };
        if (v_thread) {
            fetch_v(0, first_node(0));
            fetch_v(1, first_node(1));
        }
        bool gave_up = false;
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF, L = kk & 1;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            unsigned char *gp = smem + C::OFF_GP + L * C::GP_BYTES;
            const float4 *Ap4 = reinterpret_cast<const float4 *>(gp + C::GP_AP);
            const float4 *Pp4 = reinterpret_cast<const float4 *>(gp + C::GP_PP);
            const float4 *scal = reinterpret_cast<const float4 *>(gp + C::GP_SCAL);
            const int v_lo_next = v_thread ? first_node(kk + 2) : 0;  // needed only after this item's rows
            if (!ptx::mbar_wait(&lists_ready[L], (kk >> 1) & 1)) {
                gave_up = true;
                break;
            }
            const int n = meta_nlo(mt)[0];  // (the Gram warps read the meta block before they signalled)
            if (n > 0 && tt < 2 * NP && i < n) {
                const bool deep = meta_nlo(mt)[2] != 0;
                const unsigned char *dl = C::BIG ? s0_of(kk) : stage + C::OFF_DAP;  // full-length lists (deep trees)
                const float *Ap = reinterpret_cast<const float *>(dl);
                const float *Pp = reinterpret_cast<const float *>(dl + NP * NP * 4);
                const unsigned char *idx = C::BIG ? gp + C::GP_AP : dl + 2 * NP * NP * 4;
                float *xr = reinterpret_cast<float *>(stage + C::OFF_XR);  // (up to 32 nodes)
                const int dp = m_popc((mask_t)meta_mask(mt)[i]) - 1;  // ancestors of node i
                    const float top = wrow ? scal[i].w : 1.f;
                    unsigned char *Mhi = stage + (wrow ? C::OFF_W_HI : C::OFF_T_HI);
                    unsigned char *Mlo = stage + (wrow ? C::OFF_W_LO : C::OFF_T_LO);
                    auto put = [&](int off, float val) {  // val = hi + lo + 2^-18 |val|, both parts bf16
                        const __nv_bfloat16 hi = __float2bfloat16_rn(val);
                        *reinterpret_cast<__nv_bfloat16 *>(Mhi + off) = hi;
                        *reinterpret_cast<__nv_bfloat16 *>(Mlo + off) = __float2bfloat16_rn(val - __bfloat162float(hi));
                    };
                    if (!deep) {  // registers only, no branches: entries beyond the path are zeros
                        const uint32_t iw0 = meta_idx(mt)[i], iw1 = meta_idx(mt)[NP + i];
                        int jf[9];
                        float x[9], pe[8], co[9][8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int j = ((e < 4 ? iw0 : iw1) >> (8 * (e & 3))) & 255u;
                            jf[e] = e < dp ? j : i;
                            x[e] = 0.f;
                        }
                        jf[8] = i, x[8] = dp == 8 ? top : 0.f;
                        {
                            const float4 p0 = Pp4[i], p1 = Pp4[NP + i];
                            pe[0] = p0.x, pe[1] = p0.y, pe[2] = p0.z, pe[3] = p0.w;
                            pe[4] = p1.x, pe[5] = p1.y, pe[6] = p1.z, pe[7] = p1.w;
                        }
#pragma unroll
                        for (int f = 1; f < 9; ++f) {  // A-list of the path node at depth f
                            const float4 c0 = Ap4[jf[f]];
                            co[f][0] = c0.x, co[f][1] = c0.y, co[f][2] = c0.z, co[f][3] = c0.w;
                            if (f > 4) {
                                const float4 c1 = Ap4[NP + jf[f]];
                                co[f][4] = c1.x, co[f][5] = c1.y, co[f][6] = c1.z, co[f][7] = c1.w;
                            }
                        }
                        // x_f = 0 beyond the path, so the lists of the padding entries (node i itself)
                        // contribute nothing; only the diagonal entry e = dp must keep its value
#pragma unroll
                        for (int e = 7; e >= 0; --e) {
                            float acc = wrow ? pe[e] : 0.f;
#pragma unroll
                            for (int f = e + 1; f < 9; ++f) acc = fmaf(-x[f], co[f][e], acc);
                            x[e] = e == dp ? top : acc;
                        }
                        // entries beyond the path all aim at the diagonal and carry 0; going down from
                        // e = 8 the real diagonal entry (e = dp) is written after them
#pragma unroll
                        for (int e = 8; e >= 0; --e) {
                            put(tile_off(i, jf[e]), x[e]);
                        }
                    } else {  // deep paths: the same recurrence through shared memory (64 nodes: local memory)
                        float xloc[C::BIG ? NP : 1];
                        float *x = C::BIG ? xloc : xr + (wrow ? i : NP + i) * C::XLD;
                        auto xi = [](int e) { return e; };
                        x[xi(dp)] = top;
#pragma unroll 1
                        for (int e = dp - 1; e >= 0; --e) {
                            const int col_e = ((e >> 2) * NP) * 4 + (e & 3);
                            float acc = wrow ? Pp[col_e + i * 4] : 0.f;
#pragma unroll 1
                            for (int f = e + 1; f <= dp; ++f) {
                                const int jf = (f == dp) ? i : idx[((f >> 2) * NP + i) * 4 + (f & 3)];
                                acc = fmaf(-x[xi(f)], Ap[col_e + jf * 4], acc);
                            }
                            x[xi(e)] = acc;
                        }
#pragma unroll 1
                        for (int e = 0; e <= dp; ++e) {
                            const int col = (e == dp) ? i : idx[((e >> 2) * NP + i) * 4 + (e & 3)];
                            put(tile_off(i, col), x[xi(e)]);
                        }
                    }
            }
            ptx::fence_proxy_async();  // operand tiles were written by ordinary stores
            ptx::mbar_arrive_warp(&lists_free[L]);
            ptx::mbar_arrive_warp(&ops_ready[buf]);
            if (v_thread && !gave_up) {  // (no break: the warp's other lanes go on and meet this one at the next arrival)
                if (ptx::mbar_wait(&v_free[L], (kk >> 1) & 1)) fetch_v(kk + 2, v_lo_next);
                else gave_up = true;
            }
        }
        // after a give-up a fetch may still be in flight: it must land before the CTA exits
        if (v_thread && gave_up) {
            for (int q = 0; q < 2; ++q)
                if (v_pending[q] >= 0) ptx::mbar_wait(&v_ready[q], (v_pending[q] >> 1) & 1);
        }
    } else if (warp >= C::R_WARP0 && warp < C::E_WARP0) {
        // ------------------------------------------------------------------ R^T warps
        // Thread c = TMEM lane c = row c of d_v.  Row c of R^T, r_j = beta_j v_j - beta_j g_j (S0 k_j),
        // goes back to tensor memory as bf16 hi / lo pairs (the A operand of stage 2); g_j (S0 q_j) in place and
        // zeros over S0 k_j are what stage 2 accumulates o_j and u_j on.
        const int t = (tid - C::R_WARP0 * 32) & 127;
        const int c_lo = ((tid - C::R_WARP0 * 32) >> 7) * (NP / C::R_GROUPS), c_hi = c_lo + NP / C::R_GROUPS;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk % C::TBUF, rb = kk % C::RBUF, L = kk & 1;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            unsigned char *mt = meta_of(kk);
            unsigned char *gp = smem + C::OFF_GP + L * C::GP_BYTES;
            const float4 *scal = reinterpret_cast<const float4 *>(gp + C::GP_SCAL);
            const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(gp + C::GP_VS);
            const uint32_t tm = tmem_base + lane_base + buf * C::TM_COLS;                 // SQ | SK
            const uint32_t tr = tmem_base + lane_base + C::TM_R0 + rb * C::TM_RCOLS;            // D2 | -
            // The Gram warps signal the scalars after they have seen stage 1 complete, read the Gram block
            // out and recorded the item's size: one wait covers all of it.
            if (!ptx::mbar_wait(&scal_ready[L], (kk >> 1) & 1)) break;
            ptx::tc_fence_after_sync();
            const int n = einfo[buf].x;
            if (!ptx::mbar_wait(&v_ready[L], (kk >> 1) & 1)) break;
            if (n > 0) {
#pragma unroll 1
                for (int c0 = c_lo; c0 < c_hi; c0 += 8) {  // (rolled: code size matters more than the loop overhead)
                    uint32_t hi[4], lo[4];
                    if (c0 < n) {
                        uint32_t sk[8], sq[8];
                        ptx::tmem_ld8(tm + NP + c0, sk);
                        ptx::tmem_ld8(tm + c0, sq);
                        float v[8];
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) v[jj] = __bfloat162float(vs[(c0 + jj) * D + t]);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) {
                            const int j = c0 + jj;
                            const float4 sc = scal[j];
                            const float val = fmaf(-sc.y, __uint_as_float(sk[jj]), sc.x * v[jj]);
                            v[jj] = j < n ? val : 0.f;  // r_j
                            sq[jj] = __float_as_uint(sc.z * __uint_as_float(sq[jj]));
                            sk[jj] = 0u;
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {  // nodes 2q, 2q + 1 share a column: the lower one in its low half
                            const float h0 = ptx::bf16_hi(v[2 * q]), h1 = ptx::bf16_hi(v[2 * q + 1]);
                            hi[q] = pack_bf16(h0, h1), lo[q] = pack_bf16(v[2 * q] - h0, v[2 * q + 1] - h1);
                        }
                        ptx::tmem_st8(tm + c0, sq);
                        ptx::tmem_st8(tm + NP + c0, sk);
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) hi[q] = 0u, lo[q] = 0u;
                    }
                    ptx::tmem_st4(tr + C::TM_RHI + c0 / 2, hi);
                    ptx::tmem_st4(tr + C::TM_RLO + c0 / 2, lo);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
            }
            ptx::mbar_arrive_warp(&v_free[L]);
            ptx::mbar_arrive_warp(&lists_free[L]);
            ptx::mbar_arrive_warp(&ops_ready[buf]);
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        // u_i and o_i leave tensor memory: coalesced predicated stores, thread c = element c of a row
        const int t = tid - C::E_WARP0 * 32;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        TOut *Og = static_cast<TOut *>(a.O);
        const int rs = a.H_v * D;  // elements between a sequence's consecutive node rows
#pragma unroll 1
        for (int kk = 0;; ++kk) {
            const int item = item_of(kk);
            if (item >= n_items) break;
            const int buf = kk % C::TBUF;
            const uint32_t tm = tmem_base + lane_base + buf * C::TM_COLS;
            if (!ptx::mbar_wait(&mma2_done[buf], (kk / C::TBUF) & 1)) {
                if (t == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
                break;
            }
            ptx::tc_fence_after_sync();
            const int2 info = einfo[buf];
            const int n = info.x;
            if (n > 0) {
                const size_t row0 = (size_t)info.y * D + t;  // (the producer left the item's first row: a modulo here is 2 % of the kernel's instructions)
                TU *Ub = static_cast<TU *>(a.U) + row0;
                TOut *Ob = Og + row0;
#pragma unroll 1
                for (int c0 = 0; c0 < n; c0 += 8) {  // (rolled: code size matters more than the loop overhead)
                    uint32_t du[8], dout[8];
                    ptx::tmem_ld8(tm + C::TM_DU + c0, du);
                    ptx::tmem_ld8(tm + C::TM_DO + c0, dout);
                    ptx::tmem_wait_ld();
                    TU *Uc = Ub + (size_t)c0 * rs;
                    TOut *Oc = Ob + (size_t)c0 * rs;
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        st_global_if(Uc + jj * rs, __uint_as_float(du[jj]), c0 + jj < n);
                        st_global_if(Oc + jj * rs, __uint_as_float(dout[jj]), c0 + jj < n);
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_warp(&tmem_free[buf]);
        }
    }

    // common exit: tensor memory goes back once every role is done with it
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == C::MMA1_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, VT_TMEM_COLS);
    }
}

namespace {

template <int NP, typename TOut, bool FUSED>
cudaError_t launch_vt(const VerifyArgs &a, const PrevRound &pv, int T, cudaStream_t stream)
{
    using C = VtCfg<NP, FUSED>;
    const long long n_items = (long long)a.B * a.H_v;
    VerifyMaps m;
    const long long n_tiles = a.state_index ? (long long)a.n_states * a.H_v : n_items;
    if (!make_verify_maps(&m, a.S0, a.q, a.k, a.v, n_tiles, T, a.H_v, a.H_qk, NP)) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = current_device_sms(&dev, &sms);
    if (e != cudaSuccess) return e;
    const bool pairs = (a.H_v / a.H_qk) % 2 == 0;  // the kernel takes heads in pairs
    const long long units = pairs ? n_items / 2 : n_items;
    const int grid = (int)(units < sms ? units : sms);
    auto go = [&](auto kernel) {
        cudaError_t e2 = ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), C::SMEM_BYTES, dev);
        if (e2 != cudaSuccess) return e2;
        return launch_dependent(kernel, dim3(grid), dim3(C::THREADS), C::SMEM_BYTES, stream, a, pv, (int)n_items, m.S0, m.Q,
                                m.K, m.V);
    };
    if constexpr (FUSED) {
        return go(verify_sm100_tc_kernel<NP, TOut, true, false, float>);  // (the fused round takes fp32 U)
    } else {
        const bool cls = a.cls_lo > 0 || a.cls_hi < a.max_nodes;  // one size class of a mixed batch
        if (a.u_half)
            return cls ? go(verify_sm100_tc_kernel<NP, TOut, false, true, __half>)
                       : go(verify_sm100_tc_kernel<NP, TOut, false, false, __half>);
        return cls ? go(verify_sm100_tc_kernel<NP, TOut, false, true, float>)
                   : go(verify_sm100_tc_kernel<NP, TOut, false, false, float>);
    }
}

template <bool FUSED>
cudaError_t launch_small(const VerifyArgs &a, const PrevRound &pv, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.max_nodes <= 16)
        return od == TREEWY_F32 ? launch_vt<16, float, FUSED>(a, pv, T, stream)
                                : launch_vt<16, __nv_bfloat16, FUSED>(a, pv, T, stream);
    return od == TREEWY_F32 ? launch_vt<32, float, FUSED>(a, pv, T, stream)
                            : launch_vt<32, __nv_bfloat16, FUSED>(a, pv, T, stream);
}

}  // namespace

// bf16 inputs.  Batches of trees of up to 8 nodes take the small-tree kernel.  Otherwise sequences of
// up to 32 nodes take the kernel above, larger ones its 64-node instance; a batch that may hold both
// (max_nodes > 32) gets one launch per size class.
cudaError_t launch_verify_sm100(const VerifyArgs &a, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0 || T == 0) return cudaSuccess;
    if (a.max_nodes <= SMALL_MAX_NODES) return launch_verify_small(a, nullptr, T, od, stream);
    const PrevRound none = {};
    auto run = [&](int np, int lo, int hi) {
        VerifyArgs c = a;
        c.cls_lo = lo, c.cls_hi = hi;
        const bool f32 = od == TREEWY_F32;
        if (np == 16) return f32 ? launch_vt<16, float, false>(c, none, T, stream) : launch_vt<16, __nv_bfloat16, false>(c, none, T, stream);
        if (np == 32) return f32 ? launch_vt<32, float, false>(c, none, T, stream) : launch_vt<32, __nv_bfloat16, false>(c, none, T, stream);
        return f32 ? launch_vt<64, float, false>(c, none, T, stream) : launch_vt<64, __nv_bfloat16, false>(c, none, T, stream);
    };
    if (a.max_nodes <= 16) return run(16, 0, a.max_nodes);
    if (a.max_nodes <= 32) return run(32, 0, a.max_nodes);
    // (a third class for trees of up to 8 nodes, through the small-tree kernel, which takes half the time
    // per tree, or up to 16 nodes through the 16-node instance, was tried on the ragged workload: the extra
    // launch costs more than it saves)
    const cudaError_t e = run(32, 0, 32);
    return e != cudaSuccess ? e : run(64, 32, a.max_nodes);
}

// commit of the previous round + verify of this one, one kernel; this round's trees have <= 32 nodes
cudaError_t launch_commit_verify_sm100(const VerifyArgs &a, const PrevRound &pv, int T, treewy_dtype_t od,
                                       cudaStream_t stream)
{
    VerifyArgs small = a;
    small.cls_lo = 0, small.cls_hi = a.max_nodes;
    if (a.max_nodes <= SMALL_MAX_NODES && pv.max_nodes <= SMALL_MAX_NODES) return launch_verify_small(small, &pv, T, od, stream);
    return launch_small<true>(small, pv, T, od, stream);
}

}  // namespace treewy
