// Trees of more than 64 nodes (up to TREEWY_MAX_NODES_WIDE = 128): prepare, and the fp32 paths of verify
// (Eq. 2 and the read-out) and commit (Eq. 3), without ancestor masks.  A 64-bit mask per node is what
// the main calls key everything on; here a node's root path is walked through the parent array in
// shared memory instead, which any tree size allows.  bf16 inputs do not come here: their verify is
// the tensor-core kernel of verify_wide_tc.cu and their commit the bulk-copy pipeline of
// commit_pipe.cu.  The verify and commit kernels below are plain fp32 SIMT kernels, one CTA per
// (sequence, value head), the path fp32 inputs take.
//
//   prepare: depth and a two-word ancestor mask by walking up; L[i,h] = sum of logf(alpha[j,h]) over the
//     mask's bits in ascending node order (the order of the main prepare); level order by rank; the
//     masks stay in shared memory.
//   verify, thread c = row c of S0 (kept in registers) = element c of every u_i, o_i:
//     for node i in index order (parents first):  sk = S0[c,:].k_i, sq = S0[c,:].q_i;
//     the warps share out the ancestors j of i and reduce k_j.k_i and k_j.q_i over the lanes;
//     u_i[c] = beta_i (v_i[c] - g_i sk) - sum_j beta_i (g_i/g_j)(k_j.k_i) u_j[c],
//     o_i[c] = g_i sq + sum_{j or i} (g_i/g_j)(k_j.q_i) u_j[c];  u rows stay in shared memory.
//   commit: the accepted node's path is collected by walking up, then the tile is updated in
//     ascending path order, acc = g_a S; acc = fma(u_p[r], w_p k_p[c], acc), one rounding.
#include "treewy_common.cuh"
#include "treewy_kernels.cuh"

namespace treewy {

namespace {

constexpr int WN = TREEWY_MAX_NODES_WIDE;
constexpr int WT = 128;  // threads of a verify / prepare CTA

constexpr int WP_HCHUNK = 8;  // value heads per CTA of the prepare kernel (small: the kernel is latency bound and wants many CTAs)

// One CTA per (sequence, chunk of heads).  Node i walks up its root path through the parent array in
// shared memory for its depth and a two-word ancestor-or-self mask (kept in shared memory only: the
// wide calls hand no masks to the caller); meanwhile all threads turn the chunk's gates into
// logf(alpha).  L[i,h] is then the sum of the table's entries over the mask's bits in ascending node
// order -- the order of the main prepare, so the two agree bit for bit on trees both accept -- with
// every (i, h) independent of the others.
__global__ void __launch_bounds__(WT)
prepare_wide_kernel(int B, int T, int H_v, int max_nodes, const int32_t *__restrict__ node_offsets,
                    const int32_t *__restrict__ parent, const float *__restrict__ alpha, int32_t *__restrict__ depth,
                    float *__restrict__ cum_log_gate, uint8_t *__restrict__ level_order, int32_t *__restrict__ seq_status)
{
    __shared__ int s_bad;
    __shared__ int32_t s_parent[WN];
    __shared__ int32_t s_depth[WN];
    __shared__ unsigned long long s_mask[WN][2];
    __shared__ float s_log[WN * WP_HCHUNK];
    const int b = blockIdx.x, h0 = blockIdx.y * WP_HCHUNK;
    const int hc = min(WP_HCHUNK, H_v - h0);
    const int lo = node_offsets[b];
    const int n = node_offsets[b + 1] - lo;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const int bad = validate_sequence(parent, lo, n, T, max_nodes, &s_bad);
    if (bad) {
        if (threadIdx.x == 0 && blockIdx.y == 0 && seq_status) atomicOr(&seq_status[b], bad);
        return;
    }
    for (int i = threadIdx.x; i < n; i += WT) s_parent[i] = parent[lo + i];
    for (int e = threadIdx.x; e < n * hc; e += WT) {
        const int i = e / hc, h = e - i * hc;
        s_log[i * WP_HCHUNK + h] = logf(alpha[(size_t)(lo + i) * H_v + h0 + h]);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += WT) {
        unsigned long long m0 = 0ull, m1 = 0ull;
        int d = -1;
        for (int p = i; p >= 0; p = s_parent[p]) {  // parent[p] < p: ends
            if (p < 64) m0 |= 1ull << p;
            else m1 |= 1ull << (p - 64);
            ++d;
        }
        s_depth[i] = d;
        s_mask[i][0] = m0, s_mask[i][1] = m1;
        if (blockIdx.y == 0) depth[lo + i] = d;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n * hc; e += WT) {
        const int i = e / hc, h = e - i * hc;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            unsigned long long m = s_mask[i][w];
            while (m) {
                const int j = 64 * w + __ffsll((long long)m) - 1;
                m &= m - 1;
                acc += s_log[j * WP_HCHUNK + h];
            }
        }
        cum_log_gate[(size_t)(lo + i) * H_v + h0 + h] = acc;
    }
    if (blockIdx.y != 0) return;
    for (int i = threadIdx.x; i < n; i += WT) {
        const int di = s_depth[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const int dj = s_depth[j];
            rank += (dj < di) || (dj == di && j < i);
        }
        level_order[lo + rank] = (uint8_t)i;
    }
}

__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }

template <typename TIn> struct WideSmem {
    alignas(16) TIn kf[WN][D];     // k rows of the sequence (this head's q/k head), as stored: bf16 rows
                                   // leave room for two CTAs per SM
    float uf[WN][D];   // pseudo-values computed so far
    alignas(16) float qrow[D];  // q_i of the node being worked on
    float L[WN], beta[WN];
    int32_t parent[WN];
    float a_ij[WN], p_ij[WN];  // coefficients of node i's ancestors, in walk order (nearest first)
    int32_t anc[2][WN];        // ... and who they are (two lists: consecutive nodes alternate)
    int bad;
};

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(WT) verify_wide_kernel(VerifyArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WideSmem<TIn> &sm = *reinterpret_cast<WideSmem<TIn> *>(smem_raw);
    const int h = blockIdx.x, b = blockIdx.y;
    const int c = threadIdx.x, lane = c & 31, warp = c >> 5;
    const int lo = a.node_offsets[b];
    const int n = a.node_offsets[b + 1] - lo;
    if (c == 0) sm.bad = 0;
    __syncthreads();
    const int bad = validate_sequence(a.parent, lo, n, a.T, a.max_nodes, &sm.bad);
    if (bad) {
        if (c == 0 && h == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
        return;
    }
    for (int i = c; i < n; i += WT) sm.parent[i] = a.parent[lo + i];
    const int hq = h / (a.H_v / a.H_qk);
    const TIn *qg = static_cast<const TIn *>(a.q), *kg = static_cast<const TIn *>(a.k), *vg = static_cast<const TIn *>(a.v);
    for (int i = 0; i < n; ++i) sm.kf[i][c] = kg[((size_t)(lo + i) * a.H_qk + hq) * D + c];
    for (int i = c; i < n; i += WT) {
        sm.L[i] = a.cum_log_gate[(size_t)(lo + i) * a.H_v + h];
        sm.beta[i] = a.beta[(size_t)(lo + i) * a.H_v + h];
    }
    float srow[D];  // row c of S0
    load_row128(static_cast<const TIn *>(a.S0) + ((size_t)b * a.H_v + h) * D * D + (size_t)c * D, srow);
    __syncthreads();

    TOut *Og = static_cast<TOut *>(a.O);
    // (element c of the next node's q and v rows is fetched while the current node is worked on: one
    // CTA of four warps has nothing else to hide a global load behind)
    float q_next = to_f32(qg[((size_t)lo * a.H_qk + hq) * D + c]);
    float v_next = to_f32(vg[((size_t)lo * a.H_v + h) * D + c]);
    for (int i = 0; i < n; ++i) {
        sm.qrow[c] = q_next;
        const float v_cur = v_next;
        if (i + 1 < n) {
            q_next = to_f32(qg[((size_t)(lo + i + 1) * a.H_qk + hq) * D + c]);
            v_next = to_f32(vg[((size_t)(lo + i + 1) * a.H_v + h) * D + c]);
        }
        // ancestors of i, nearest first (every thread walks the same chain: no divergence)
        int32_t *anc = sm.anc[i & 1];  // (slower threads may still read the previous node's list)
        int na = 0;
        for (int p = sm.parent[i]; p >= 0; p = sm.parent[p]) {
            if (c == 0) anc[na] = p;
            ++na;
        }
        __syncthreads();  // q_i and the ancestor list are in place (and the previous node's coefficients are read)
        // k_j . k_i and k_j . q_i: warp w takes ancestors w, w + 4, ..., lanes share the 128 elements
        const float Li = sm.L[i], bi = sm.beta[i];
        for (int e = warp; e <= na; e += WT / 32) {  // e == na: the node itself (q_i . k_i)
            const int j = e < na ? anc[e] : i;
            float kk = 0.f, qk = 0.f;
#pragma unroll
            for (int t = 0; t < D / 32; ++t) {
                const float kj = to_f32(sm.kf[j][lane + 32 * t]);
                kk = fmaf(kj, to_f32(sm.kf[i][lane + 32 * t]), kk);
                qk = fmaf(kj, sm.qrow[lane + 32 * t], qk);
            }
            kk = warp_sum(kk), qk = warp_sum(qk);
            if (lane == 0) {
                const float ratio = expf(Li - sm.L[j]);
                sm.a_ij[e] = bi * ratio * kk;  // (unused for e == na)
                sm.p_ij[e] = ratio * qk;
            }
        }
        // S0 k_i and S0 q_i for this thread's row
        float sk0 = 0.f, sk1 = 0.f, sq0 = 0.f, sq1 = 0.f;
#pragma unroll
        for (int d = 0; d < D; d += 4) {
            const float4 k4 = load4(&sm.kf[i][d]);
            const float4 q4 = *reinterpret_cast<const float4 *>(&sm.qrow[d]);
            sk0 = fmaf(srow[d], k4.x, sk0), sk1 = fmaf(srow[d + 1], k4.y, sk1);
            sk0 = fmaf(srow[d + 2], k4.z, sk0), sk1 = fmaf(srow[d + 3], k4.w, sk1);
            sq0 = fmaf(srow[d], q4.x, sq0), sq1 = fmaf(srow[d + 1], q4.y, sq1);
            sq0 = fmaf(srow[d + 2], q4.z, sq0), sq1 = fmaf(srow[d + 3], q4.w, sq1);
        }
        __syncthreads();  // the coefficients are written
        const float g = expf(Li);
        const size_t orow = ((size_t)(lo + i) * a.H_v + h) * D + c;
        float u = bi * (v_cur - g * (sk0 + sk1));
        float o = g * (sq0 + sq1);
        for (int e = na - 1; e >= 0; --e) {  // ascending node index: root first
            const float uj = sm.uf[anc[e]][c];
            u = fmaf(-sm.a_ij[e], uj, u);
            o = fmaf(sm.p_ij[e], uj, o);
        }
        o = fmaf(sm.p_ij[na], u, o);
        sm.uf[i][c] = u;  // read back only by this thread
        store_u(a.U, orow, u, a.u_half);
        Og[orow] = from_f32<TOut>(o);
    }
}

constexpr int WC_THREADS = 256;

// one CTA per (sequence, value head); thread (r0, cc): rows r0, r0 + 16, ..., columns 8 cc .. 8 cc + 7
template <typename T> __global__ void __launch_bounds__(WC_THREADS) commit_wide_kernel(CommitArgs a)
{
    __shared__ int s_bad;
    __shared__ int32_t s_parent[WN];
    __shared__ int32_t s_path[WN];
    __shared__ float s_w[WN];
    const int h = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, cc = tid & 15, r0 = tid >> 4;
    const int lo = a.node_offsets[b];
    const int n = a.node_offsets[b + 1] - lo;
    if (tid == 0) s_bad = 0;
    __syncthreads();
    int bad = validate_sequence(a.parent, lo, n, a.T, a.max_nodes, &s_bad);
    const int acc_node = a.accepted[b];
    if (!bad && (acc_node < -1 || acc_node >= n)) bad = TREEWY_SEQ_BAD_ACCEPTED;
    if (bad) {
        if (tid == 0 && h == 0 && a.seq_status) atomicOr(&a.seq_status[b], bad);
        return;
    }
    if (acc_node < 0 && !a.S_out_f32) return;  // the state stays as it is

    T *Sg = static_cast<T *>(a.S0) + ((size_t)b * a.H_v + h) * D * D;
    float acc[8][8];
#pragma unroll
    for (int it = 0; it < 8; ++it)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[it][e] = to_f32(Sg[(size_t)(r0 + 16 * it) * D + cc * 8 + e]);

    if (acc_node >= 0) {
        for (int i = tid; i < n; i += WC_THREADS) s_parent[i] = a.parent[lo + i];
        __syncthreads();
        int plen = 0;
        for (int p = acc_node; p >= 0; p = s_parent[p]) ++plen;  // every thread: the same walk
        const float La = a.cum_log_gate[(size_t)(lo + acc_node) * a.H_v + h];
        if (tid == 0) {
            int e = plen;
            for (int p = acc_node; p >= 0; p = s_parent[p]) s_path[--e] = p;  // ascending: root first
        }
        __syncthreads();
        for (int e = tid; e < plen; e += WC_THREADS)
            s_w[e] = expf(La - a.cum_log_gate[(size_t)(lo + s_path[e]) * a.H_v + h]);
        __syncthreads();
        const float ga = expf(La);
#pragma unroll
        for (int it = 0; it < 8; ++it)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[it][e] *= ga;
        const int hq = h / (a.H_v / a.H_qk);
        const T *kg = static_cast<const T *>(a.k);
        for (int e = 0; e < plen; ++e) {
            const int j = s_path[e];
            const float w = s_w[e];
            float kf[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) kf[x] = to_f32(kg[((size_t)(lo + j) * a.H_qk + hq) * D + cc * 8 + x]) * w;
            const size_t ur = ((size_t)(lo + j) * a.H_v + h) * D;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const float u = load_u(a.U, ur + r0 + 16 * it, a.u_half);
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[it][x] = fmaf(u, kf[x], acc[it][x]);
            }
        }
#pragma unroll
        for (int it = 0; it < 8; ++it)
#pragma unroll
            for (int e = 0; e < 8; ++e) Sg[(size_t)(r0 + 16 * it) * D + cc * 8 + e] = from_f32<T>(acc[it][e]);
    }
    if (a.S_out_f32) {
        float *o = a.S_out_f32 + ((size_t)b * a.H_v + h) * D * D;
#pragma unroll
        for (int it = 0; it < 8; ++it)
#pragma unroll
            for (int e = 0; e < 8; ++e) o[(size_t)(r0 + 16 * it) * D + cc * 8 + e] = acc[it][e];
    }
}

}  // namespace

cudaError_t launch_prepare_wide(const treewy_tree_t &t, int max_nodes, const float *alpha, int32_t *seq_status,
                                cudaStream_t stream)
{
    if (t.B == 0) return cudaSuccess;
    prepare_wide_kernel<<<dim3(t.B, (t.H_v + WP_HCHUNK - 1) / WP_HCHUNK), WT, 0, stream>>>(t.B, t.T, t.H_v, max_nodes, t.node_offsets, t.parent, alpha, t.depth,
                                                t.cum_log_gate, t.level_order, seq_status);
    return cudaGetLastError();
}

template <typename TIn, typename TOut> static cudaError_t launch_vw(const VerifyArgs &a, cudaStream_t stream)
{
    const int smem = (int)sizeof(WideSmem<TIn>);
    cudaError_t e = cudaFuncSetAttribute(verify_wide_kernel<TIn, TOut>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    verify_wide_kernel<TIn, TOut><<<dim3(a.H_v, a.B), WT, smem, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_verify_wide(const VerifyArgs &a, treewy_dtype_t io, treewy_dtype_t od, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0) return cudaSuccess;
    if (io == TREEWY_BF16) return launch_verify_wide_tc(a, od, stream);  // TMA + tcgen05
    return od == TREEWY_F32 ? launch_vw<float, float>(a, stream) : launch_vw<float, __nv_bfloat16>(a, stream);
}

cudaError_t launch_commit_wide(const CommitArgs &a, treewy_dtype_t io, cudaStream_t stream)
{
    if (a.B == 0 || a.H_v == 0) return cudaSuccess;
    if (io == TREEWY_BF16) return launch_commit_pipe(a, stream);  // (no masks in `a`: the pipeline walks parents)
    commit_wide_kernel<float><<<dim3(a.H_v, a.B), WC_THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace treewy
