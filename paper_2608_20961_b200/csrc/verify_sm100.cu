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
//   consumer warps 0-3 (128 threads; thread c owns TMEM lane c = row c of d_v)
//       scale + mask the Gram rows into the coefficient matrix
//           A[i,j] = beta_i e^{L_i-L_j} k_i.k_j  (j proper ancestor),
//           P[i,j] = e^{L_i-L_j} q_i.k_j         (j ancestor or self),
//       then every thread runs the forward substitution of (I + A) U = R for its own column,
//       walking each node's ancestor list (fp32 FMA), and reads the outputs out of the same
//       pass:  u_i = beta_i (v_i - e^{L_i} S0k_i) - sum A[i,j] u_j ,
//              o_i = e^{L_i} S0q_i + sum P[i,j] u_j .
//       tcgen05.ld hands thread c exactly column c of S0 Q^T / S0 K^T, so no value crosses
//       threads.  U (fp32) and O are stored coalesced (a warp writes 128 contiguous bytes).
//
// Every mbarrier wait is bounded; on give-up the role leaves its loop, TREEWY_SEQ_TIMEOUT is
// raised, and the CTA still reaches the common exit where tensor memory is freed.
#include <cuda.h>

#include "ptx_sm100.cuh"
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr int VS_CONSUMERS = 128;
constexpr uint32_t VS_TMEM_COLS = 512;

template <int NP> struct VsCfg {
    static constexpr int STAGES = NP <= 32 ? 3 : 2;
    static constexpr int THREADS = VS_CONSUMERS + 32 + 32 * STAGES;
    static constexpr int QK_HALF = 2 * NP * 128;  // one 64-column half of the [Q;K] rows, bytes
    static constexpr int QK_BYTES = 2 * QK_HALF;
    static constexpr int S0_HALF = D * 128;
    static constexpr int S0_BYTES = 2 * S0_HALF;
    static constexpr int V_BYTES = NP * D * 2;
    static constexpr int OFF_S0 = QK_BYTES;
    static constexpr int OFF_V = OFF_S0 + S0_BYTES;
    static constexpr int OFF_META = OFF_V + V_BYTES;
    static constexpr int META_BYTES = NP * 16 + 16;  // mask u64, L f32, beta f32 per node; n, lo
    static constexpr int STAGE_BYTES = (OFF_META + META_BYTES + 1023) / 1024 * 1024;
    static constexpr int LD = NP + 1;  // row stride of the coefficient matrix
    static constexpr int OFF_US = STAGES * STAGE_BYTES;
    static constexpr int OFF_COEF = OFF_US + NP * D * 4;
    static constexpr int OFF_GS = OFF_COEF + NP * LD * 4;
    static constexpr int OFF_BAR = (OFF_GS + NP * 4 + 15) / 16 * 16;
    static constexpr int SMEM_BYTES = OFF_BAR + (2 * STAGES + 4) * 8 + 16 + 1024;  // + align slack
    static constexpr uint32_t TX_BYTES = S0_BYTES + QK_BYTES + V_BYTES;
};

struct VsMeta {  // view of a stage's meta block
    unsigned long long *mask;
    float *L, *beta;
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
    float *us = reinterpret_cast<float *>(smem + C::OFF_US);
    float *coef = reinterpret_cast<float *>(smem + C::OFF_COEF);
    float *gs = reinterpret_cast<float *>(smem + C::OFF_GS);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint64_t *empty = full + C::STAGES;
    uint64_t *mma_done = empty + C::STAGES;
    uint64_t *tmem_free = mma_done + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tmem_free + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int MMA_WARP = VS_CONSUMERS / 32;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], VS_CONSUMERS);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&mma_done[i], 1);
            ptx::mbar_init(&tmem_free[i], VS_CONSUMERS);
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
            if (n < 1 || n > a.max_nodes || n > NP) {
                bad = TREEWY_SEQ_TOO_MANY_NODES;
            } else {
                int bp = 0;
                for (int i = lane; i < n; i += 32) {
                    const int p = a.parent[lo + i];
                    bp |= (p < -1 || p >= i);
                }
                if (__any_sync(0xffffffffu, bp)) bad = TREEWY_SEQ_BAD_PARENT;
            }
            if (bad && h == 0 && lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
            // node scalars: issued before the wait so their latency hides under it
            unsigned long long mk[(NP + 31) / 32];
            float Lv[(NP + 31) / 32], bv[(NP + 31) / 32];
#pragma unroll
            for (int r = 0; r < (NP + 31) / 32; ++r) {
                const int i = lane + 32 * r;
                const bool on = !bad && i < n;
                mk[r] = on ? a.anc_mask[lo + i] : 0ull;
                Lv[r] = on ? a.cum_log_gate[(size_t)(lo + i) * a.H_v + h] : 0.f;
                bv[r] = on ? a.beta[(size_t)(lo + i) * a.H_v + h] : 0.f;
            }
            if (!ptx::mbar_wait(&empty[s], ((kk / C::STAGES) & 1) ^ 1)) {
                if (lane == 0 && a.seq_status) atomicOr(&a.seq_status[b], TREEWY_SEQ_TIMEOUT);
                break;
            }
#pragma unroll
            for (int r = 0; r < (NP + 31) / 32; ++r) {
                const int i = lane + 32 * r;
                if (i < NP) mt.mask[i] = mk[r], mt.L[i] = Lv[r], mt.beta[i] = bv[r];
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
            const int s = kk % C::STAGES, buf = kk & 1;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            if (!ptx::mbar_wait(&full[s], (kk / C::STAGES) & 1)) break;
            const int n = vs_meta<NP>(stage).n_lo[0];
            if (!ptx::mbar_wait(&tmem_free[buf], ((kk >> 1) & 1) ^ 1)) break;
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
        TOut *Og = static_cast<TOut *>(a.O);
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        for (int kk = 0;; ++kk) {
            const int item = blockIdx.x + kk * gridDim.x;
            if (item >= n_items) break;
            const int s = kk % C::STAGES, buf = kk & 1;
            unsigned char *stage = smem + s * C::STAGE_BYTES;
            if (!ptx::mbar_wait(&mma_done[buf], (kk >> 1) & 1)) {
                if (tid == 0 && a.seq_status) atomicOr(&a.seq_status[item / a.H_v], TREEWY_SEQ_TIMEOUT);
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

                ptx::named_sync(1, VS_CONSUMERS);  // previous item's coefficient reads are over
                {   // Gram rows -> scaled, masked coefficients
                    const bool p_row = tid < n;                      // q_i . k_j, i = tid
                    const bool a_row = tid >= NP && tid - NP < n;    // k_i . k_j, i = tid - NP
                    const int i = p_row ? tid : tid - NP;
                    const bool mine = p_row || a_row;
                    const unsigned long long mi = mine ? mt.mask[i] : 0ull;
                    const float Li = mine ? mt.L[i] : 0.f;
                    const float scale = a_row ? mt.beta[i] : 1.f;
                    if (p_row) gs[i] = expf(Li);
#pragma unroll
                    for (int c0 = 0; c0 < NP; c0 += 16) {
                        if (c0 < n) {
                            uint32_t g[16];
                            ptx::tmem_ld16(d2 + c0, g);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) {
                                const int j = c0 + jj;
                                if ((mi >> j) & 1ull) {
                                    const float val = scale * expf(Li - mt.L[j]) * __uint_as_float(g[jj]);
                                    if (p_row) coef[j * C::LD + i + 1] = val;
                                    else if (j != i) coef[i * C::LD + j] = val;
                                }
                            }
                        }
                    }
                }
                ptx::named_sync(1, VS_CONSUMERS);

#pragma unroll
                for (int c0 = 0; c0 < NP; c0 += 16) {
                    if (c0 < n) {
                        uint32_t sq[16], sk[16];
                        ptx::tmem_ld16(d1 + c0, sq);
                        ptx::tmem_ld16(d1 + NP + c0, sk);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int ii = 0; ii < 16; ++ii) {
                            const int i = c0 + ii;
                            if (i < n) {
                                const float g = gs[i];
                                const float v = __bfloat162float(vs[i * D + tid]);
                                float u = mt.beta[i] * (v - g * __uint_as_float(sk[ii]));
                                float o = g * __uint_as_float(sq[ii]);
                                unsigned long long m = mt.mask[i] & ~(1ull << i);
                                while (m) {
                                    const int j = __ffsll((long long)m) - 1;
                                    m &= m - 1;
                                    const float uj = us[j * D + tid];
                                    u = fmaf(-coef[i * C::LD + j], uj, u);
                                    o = fmaf(coef[j * C::LD + i + 1], uj, o);
                                }
                                o = fmaf(coef[i * C::LD + i + 1], u, o);
                                us[i * D + tid] = u;
                                const size_t row = ((size_t)(lo + i) * a.H_v + h) * D + tid;
                                a.U[row] = u;
                                Og[row] = from_f32<TOut>(o);
                            }
                        }
                    }
                }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// bf16 matrix [rows, cols] with `row_bytes` between rows; box = box_cols x box_rows
bool make_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows,
              uint64_t row_bytes, uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw)
{
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NP, typename TOut>
cudaError_t launch_vs(const VerifyArgs &a, int T, cudaStream_t stream)
{
    using C = VsCfg<NP>;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const long long n_items = (long long)a.B * a.H_v;
    CUtensorMap tmS0, tmQ, tmK, tmV;
    bool ok = make_map(enc, &tmS0, a.S0, D, (uint64_t)n_items * D, D * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && make_map(enc, &tmQ, a.q, (uint64_t)a.H_qk * D, T, (uint64_t)a.H_qk * D * 2, 64, NP,
                        CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && make_map(enc, &tmK, a.k, (uint64_t)a.H_qk * D, T, (uint64_t)a.H_qk * D * 2, 64, NP,
                        CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && make_map(enc, &tmV, a.v, (uint64_t)a.H_v * D, T, (uint64_t)a.H_v * D * 2, 128, NP,
                        CU_TENSOR_MAP_SWIZZLE_NONE);
    if (!ok) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(verify_sm100_kernel<NP, TOut>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int grid = (int)(n_items < sms ? n_items : sms);
    verify_sm100_kernel<NP, TOut><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(a, (int)n_items, tmS0, tmQ,
                                                                                tmK, tmV);
    return cudaGetLastError();
}

template <typename TOut> cudaError_t launch_vs_np(const VerifyArgs &a, int T, cudaStream_t stream)
{
    if (a.max_nodes <= 16) return launch_vs<16, TOut>(a, T, stream);
    if (a.max_nodes <= 32) return launch_vs<32, TOut>(a, T, stream);
    return launch_vs<64, TOut>(a, T, stream);
}

}  // namespace

cudaError_t launch_verify_sm100(const VerifyArgs &a, int T, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0 || T == 0) return cudaSuccess;
    if (od == TREEWY_F32) return launch_vs_np<float>(a, T, stream);
    return launch_vs_np<__nv_bfloat16>(a, T, stream);
}

}  // namespace treewy
