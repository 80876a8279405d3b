// treewy_commit: rebuild the accepted node's state in place (Section 3, Eq. 3):
//     S_a = g_a S0 + sum_{j ancestor-or-self of a} (g_a / g_j) u_j k_j^T .
//
// A pure streaming kernel: every state element is read once, gets <= depth+1 rank-1 terms in
// fp32, is rounded once and written back to the same address (each element depends only on
// itself, so updating in place is safe).  One CTA of 256 threads owns a slab of
// 16*RPT rows x 128 columns of one (sequence, value head) state; a thread owns an 8-column
// chunk (16 bytes of bf16) of RPT rows.  The state loads are issued first, the short
// dependent chain  accepted -> ancestor mask -> log-gates -> k / U rows  runs under them, and
// the path's rows are staged through shared memory eight nodes at a time:
//     kw[p][c] = e^{L_a - L_j} k_j[c]   (gate ratio folded into the key row),
//     uu[p][r] = u_j[r] .
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

constexpr int CM_THREADS = 256;
constexpr int CM_PCH = 8;  // path nodes staged per pass

template <typename T> struct Raw8;  // eight consecutive state elements as loaded
template <> struct Raw8<__nv_bfloat16> {
    uint4 x;
    __device__ __forceinline__ void load(const __nv_bfloat16 *p) { x = *reinterpret_cast<const uint4 *>(p); }
    __device__ __forceinline__ void widen(float (&f)[8]) const
    {
        f[0] = bf16lo(x.x), f[1] = bf16hi(x.x), f[2] = bf16lo(x.y), f[3] = bf16hi(x.y);
        f[4] = bf16lo(x.z), f[5] = bf16hi(x.z), f[6] = bf16lo(x.w), f[7] = bf16hi(x.w);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&f)[8])
    {
        uint4 y;
        y.x = pack_bf16(f[0], f[1]), y.y = pack_bf16(f[2], f[3]);
        y.z = pack_bf16(f[4], f[5]), y.w = pack_bf16(f[6], f[7]);
        *reinterpret_cast<uint4 *>(p) = y;
    }
};
template <> struct Raw8<float> {
    float4 x, y;
    __device__ __forceinline__ void load(const float *p)
    {
        x = reinterpret_cast<const float4 *>(p)[0];
        y = reinterpret_cast<const float4 *>(p)[1];
    }
    __device__ __forceinline__ void widen(float (&f)[8]) const
    {
        f[0] = x.x, f[1] = x.y, f[2] = x.z, f[3] = x.w, f[4] = y.x, f[5] = y.y, f[6] = y.z, f[7] = y.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&f)[8])
    {
        reinterpret_cast<float4 *>(p)[0] = make_float4(f[0], f[1], f[2], f[3]);
        reinterpret_cast<float4 *>(p)[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
};

template <typename T, int RPT>
__global__ void __launch_bounds__(CM_THREADS) commit_kernel(CommitArgs a)
{
    constexpr int ROWS = 16 * RPT;       // rows of the slab
    constexpr int SLABS = D / ROWS;      // slabs per state
    __shared__ __align__(16) float kw[CM_PCH][D];
    __shared__ float uu[CM_PCH][ROWS];
    __shared__ int s_bad;

    const int h = blockIdx.x / SLABS, slab = blockIdx.x % SLABS, b = blockIdx.y;
    const int tid = threadIdx.x;
    const int cc = tid & 15, r0 = tid >> 4;
    const int lo = a.node_offsets[b];
    const int n = a.node_offsets[b + 1] - lo;
    const int acc_node = a.accepted[b];

    const int slot = state_slot(a.state_index, a.n_states, b);
    T *tile = static_cast<T *>(a.S0) + ((size_t)(slot < 0 ? 0 : slot) * a.H_v + h) * D * D + (size_t)slab * ROWS * D;
    float *tile32 =
        a.S_out_f32 ? a.S_out_f32 + ((size_t)b * a.H_v + h) * D * D + (size_t)slab * ROWS * D : nullptr;

    if (tid == 0) s_bad = 0;
    __syncthreads();
    int bad = validate_sequence(a.parent, lo, n, a.T, a.max_nodes, &s_bad);
    if (!bad && (acc_node < -1 || acc_node >= n)) bad = TREEWY_SEQ_BAD_ACCEPTED;
    if (slot < 0) bad = TREEWY_SEQ_BAD_STATE;
    if (bad) {
        if (tid == 0 && blockIdx.x == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
        return;
    }
    if (acc_node < 0 && tile32 == nullptr) return;  // state stays as it is

    // the slab's state elements, in flight while the path is staged
    Raw8<T> raw[RPT];
#pragma unroll
    for (int it = 0; it < RPT; ++it) raw[it].load(tile + (size_t)(r0 + 16 * it) * D + cc * 8);

    float acc[RPT][8];
    if (acc_node < 0) {
#pragma unroll
        for (int it = 0; it < RPT; ++it) {
            raw[it].widen(acc[it]);
            Raw8<float>::store(tile32 + (size_t)(r0 + 16 * it) * D + cc * 8, acc[it]);
        }
        return;
    }

    const uint64_t path = a.anc_mask[lo + acc_node];
    const float La = a.cum_log_gate[(size_t)(lo + acc_node) * a.H_v + h];
    const int hq = h / (a.H_v / a.H_qk);
    const T *kg = static_cast<const T *>(a.k);

    bool first = true;
    uint64_t rest = path;
    while (rest) {
        // stage up to CM_PCH path nodes
        uint64_t m = rest;
        int cnt = 0;
        __syncthreads();  // previous pass has finished reading kw / uu
        for (; m && cnt < CM_PCH; ++cnt) {
            const int j = __ffsll((long long)m) - 1;
            m &= m - 1;
            const float w = expf(La - a.cum_log_gate[(size_t)(lo + j) * a.H_v + h]);
            if (tid < D)
                kw[cnt][tid] = w * to_f32(kg[((size_t)(lo + j) * a.H_qk + hq) * D + tid]);
            else if (tid - D < ROWS)
                uu[cnt][tid - D] = load_u(a.U, ((size_t)(lo + j) * a.H_v + h) * D + slab * ROWS + tid - D, a.u_half);
        }
        rest = m;
        __syncthreads();

        if (first) {
            const float ga = expf(La);
#pragma unroll
            for (int it = 0; it < RPT; ++it) {
                raw[it].widen(acc[it]);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[it][e] *= ga;
            }
            first = false;
        }
        for (int p = 0; p < cnt; ++p) {
            const float4 k0 = *reinterpret_cast<const float4 *>(&kw[p][cc * 8]);
            const float4 k1 = *reinterpret_cast<const float4 *>(&kw[p][cc * 8 + 4]);
#pragma unroll
            for (int it = 0; it < RPT; ++it) {
                const float u = uu[p][r0 + 16 * it];
                acc[it][0] = fmaf(u, k0.x, acc[it][0]);
                acc[it][1] = fmaf(u, k0.y, acc[it][1]);
                acc[it][2] = fmaf(u, k0.z, acc[it][2]);
                acc[it][3] = fmaf(u, k0.w, acc[it][3]);
                acc[it][4] = fmaf(u, k1.x, acc[it][4]);
                acc[it][5] = fmaf(u, k1.y, acc[it][5]);
                acc[it][6] = fmaf(u, k1.z, acc[it][6]);
                acc[it][7] = fmaf(u, k1.w, acc[it][7]);
            }
        }
    }
#pragma unroll
    for (int it = 0; it < RPT; ++it) {
        Raw8<T>::store(tile + (size_t)(r0 + 16 * it) * D + cc * 8, acc[it]);
        if (tile32) Raw8<float>::store(tile32 + (size_t)(r0 + 16 * it) * D + cc * 8, acc[it]);
    }
}

template <typename T, int RPT>
static cudaError_t launch_cm(const CommitArgs &a, cudaStream_t stream)
{
    dim3 grid(a.H_v * (D / (16 * RPT)), a.B);
    commit_kernel<T, RPT><<<grid, CM_THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_commit(const CommitArgs &a, treewy_dtype_t io, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0) return cudaSuccess;
    if (io == TREEWY_F32) return launch_cm<float, 4>(a, stream);
    return launch_commit_pipe(a, stream);
}

}  // namespace treewy
