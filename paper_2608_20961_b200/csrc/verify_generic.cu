// treewy_verify, portable fp32 SIMT kernel (Section 3: Eq. 2 and the read-out).
//
// One CTA of 128 threads per (sequence b, value head h).  Thread c owns row c of the state
// (the d_v index) in registers and, with it, column c of every [N x d_v] quantity: the
// triangular system (I + A) U = R has the same matrix for all 128 columns, so each thread
// runs its own forward substitution and no value ever crosses threads after the Gram step.
//
//   Gram   KK[i,j] = k_i . k_j (j a proper ancestor of i), QK[i,j] = q_i . k_j (j ancestor or
//          self): one warp per pair, only ancestor pairs are formed.  Scaled on the spot:
//          A[i,j] = beta_i e^{L_i - L_j} KK[i,j],  P[i,j] = e^{L_i - L_j} QK[i,j]
//          (L the cumulative log-gate; the exponent is <= 0 so nothing overflows).
//   node i (in index order, parents first):
//          u_i[c] = beta_i (v_i[c] - e^{L_i} (S0 k_i)[c]) - sum_{j<i anc} A[i,j] u_j[c]
//          o_i[c] = e^{L_i} (S0 q_i)[c] + sum_{j anc-or-self} P[i,j] u_j[c]
//
// Everything is fp32 FMA; inputs may be fp32 or bf16 (widened exactly on load).
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr int VG_THREADS = 128;

// shared-memory layout for a launch sized for `nmax` nodes (floats unless noted)
__host__ __device__ inline size_t vg_smem_bytes(int nmax)
{
    return (size_t)nmax * D * 4 * 3      // k rows, q rows, U
           + (size_t)nmax * nmax * 4 * 2  // A, P
           + (size_t)nmax * (8 + 4 + 4);  // mask, L, beta
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(VG_THREADS) verify_generic_kernel(VerifyArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_bad;

    const int h = blockIdx.x, b = blockIdx.y;
    const int nmax = a.max_nodes;
    const int lo = a.node_offsets[b];
    const int n = a.node_offsets[b + 1] - lo;
    const int c = threadIdx.x, lane = c & 31, warp = c >> 5;

    if (c == 0) s_bad = 0;
    __syncthreads();
    const int slot = state_slot(a.state_index, a.n_states, b);
    const int bad = slot < 0 ? TREEWY_SEQ_BAD_STATE : validate_sequence(a.parent, lo, n, a.T, nmax, &s_bad);
    if (bad) {
        if (c == 0 && h == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
        return;
    }

    float *ks = reinterpret_cast<float *>(smem_raw);
    float *qs = ks + (size_t)nmax * D;
    float *us = qs + (size_t)nmax * D;
    float *As = us + (size_t)nmax * D;
    float *Ps = As + (size_t)nmax * nmax;
    uint64_t *ms = reinterpret_cast<uint64_t *>(Ps + (size_t)nmax * nmax);
    float *Ls = reinterpret_cast<float *>(ms + nmax);
    float *bs = Ls + nmax;

    const int hq = h / (a.H_v / a.H_qk);
    const TIn *qg = static_cast<const TIn *>(a.q);
    const TIn *kg = static_cast<const TIn *>(a.k);
    const TIn *vg = static_cast<const TIn *>(a.v);

    for (int i = 0; i < n; ++i) {
        const size_t row = ((size_t)(lo + i) * a.H_qk + hq) * D;
        ks[i * D + c] = to_f32(kg[row + c]);
        qs[i * D + c] = to_f32(qg[row + c]);
    }
    if (c < n) {
        ms[c] = a.anc_mask[lo + c];
        Ls[c] = a.cum_log_gate[(size_t)(lo + c) * a.H_v + h];
        bs[c] = a.beta[(size_t)(lo + c) * a.H_v + h];
    }

    // row c of S0[b,h] into registers
    float s[D];
    {
        const TIn *srow = static_cast<const TIn *>(a.S0) + (((size_t)slot * a.H_v + h) * D + c) * D;
        load_row128(srow, s);
    }
    __syncthreads();

    // Gram entries of ancestor pairs, scaled.  Warp w takes nodes w, w+4, ...
    for (int i = warp; i < n; i += VG_THREADS / 32) {
        uint64_t m = ms[i];
        const float4 ki = *reinterpret_cast<const float4 *>(ks + i * D + lane * 4);
        const float4 qi = *reinterpret_cast<const float4 *>(qs + i * D + lane * 4);
        while (m) {
            const int j = __ffsll((long long)m) - 1;
            m &= m - 1;
            const float4 kj = *reinterpret_cast<const float4 *>(ks + j * D + lane * 4);
            float kk = ki.x * kj.x + ki.y * kj.y + ki.z * kj.z + ki.w * kj.w;
            float qk = qi.x * kj.x + qi.y * kj.y + qi.z * kj.z + qi.w * kj.w;
            kk = warp_sum(kk);
            qk = warp_sum(qk);
            if (lane == 0) {
                const float e = expf(Ls[i] - Ls[j]);
                As[i * nmax + j] = bs[i] * e * kk;
                Ps[i * nmax + j] = e * qk;
            }
        }
    }
    __syncthreads();

    TOut *Og = static_cast<TOut *>(a.O);
    for (int i = 0; i < n; ++i) {
        const float *ki = ks + i * D;
        const float *qi = qs + i * D;
        float sk0 = 0.f, sk1 = 0.f, sq0 = 0.f, sq1 = 0.f;
#pragma unroll
        for (int d = 0; d < D; d += 4) {
            const float4 kk = *reinterpret_cast<const float4 *>(ki + d);
            const float4 qq = *reinterpret_cast<const float4 *>(qi + d);
            sk0 = fmaf(s[d], kk.x, sk0);
            sk1 = fmaf(s[d + 1], kk.y, sk1);
            sk0 = fmaf(s[d + 2], kk.z, sk0);
            sk1 = fmaf(s[d + 3], kk.w, sk1);
            sq0 = fmaf(s[d], qq.x, sq0);
            sq1 = fmaf(s[d + 1], qq.y, sq1);
            sq0 = fmaf(s[d + 2], qq.z, sq0);
            sq1 = fmaf(s[d + 3], qq.w, sq1);
        }
        const float g = expf(Ls[i]);
        const size_t orow = ((size_t)(lo + i) * a.H_v + h) * D + c;
        float u = bs[i] * (to_f32(vg[orow]) - g * (sk0 + sk1));
        float o = g * (sq0 + sq1);
        uint64_t m = ms[i] & ~(1ull << i);
        while (m) {
            const int j = __ffsll((long long)m) - 1;
            m &= m - 1;
            const float uj = us[j * D + c];
            u = fmaf(-As[i * nmax + j], uj, u);
            o = fmaf(Ps[i * nmax + j], uj, o);
        }
        o = fmaf(Ps[i * nmax + i], u, o);
        us[i * D + c] = u;  // read back only by this thread: no barrier needed
        store_u(a.U, orow, u, a.u_half);
        Og[orow] = from_f32<TOut>(o);
    }
}

template <typename TIn, typename TOut>
static cudaError_t launch_vg(const VerifyArgs &a, cudaStream_t stream)
{
    const size_t smem = vg_smem_bytes(a.max_nodes);
    cudaError_t e = cudaFuncSetAttribute(verify_generic_kernel<TIn, TOut>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.H_v, a.B);
    verify_generic_kernel<TIn, TOut><<<grid, VG_THREADS, smem, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_verify_generic(const VerifyArgs &a, treewy_dtype_t io, treewy_dtype_t od,
                                  cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0) return cudaSuccess;
    if (io == TREEWY_F32 && od == TREEWY_F32) return launch_vg<float, float>(a, stream);
    if (io == TREEWY_F32 && od == TREEWY_BF16) return launch_vg<float, __nv_bfloat16>(a, stream);
    if (io == TREEWY_BF16 && od == TREEWY_F32) return launch_vg<__nv_bfloat16, float>(a, stream);
    return launch_vg<__nv_bfloat16, __nv_bfloat16>(a, stream);
}

}  // namespace treewy
