// Shared device helpers of libtreewy's kernels: storage-type conversion, per-sequence
// validation, small warp utilities.  Nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/treewy.h"

namespace treewy {

constexpr int D = TREEWY_D;
constexpr int MAXN = TREEWY_MAX_NODES;

// Programmatic dependent launch: every kernel of the library is launched so that it may become
// resident while the kernel before it on the stream is still running (its launch latency and its
// prologue then overlap that kernel's tail).  grid_dependency_wait() returns once the preceding
// kernel has finished and its writes are visible: a kernel calls it before its first access to
// global memory, whatever the buffer, since the library cannot know what the kernel before it wrote.
// grid_dependency_trigger() lets the kernel after this one become resident as resources free up.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Host side of a launch, kept off the per-call path: the SM count of a device and the raised dynamic
// shared-memory limit of a kernel are looked up / set once per device and process (on a batch of a
// few dozen microseconds of GPU work, three runtime calls per launch are a visible part of the step).
inline cudaError_t current_device_sms(int *dev, int *sms)
{
    static std::atomic<int> cache[64];
    cudaError_t e = cudaGetDevice(dev);
    if (e != cudaSuccess) return e;
    const bool cached = *dev >= 0 && *dev < 64;
    if (cached && (*sms = cache[*dev].load(std::memory_order_relaxed)) > 0) return cudaSuccess;
    e = cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, *dev);
    if (e == cudaSuccess && cached) cache[*dev].store(*sms, std::memory_order_relaxed);
    return e;
}
inline cudaError_t ensure_dynamic_smem(const void *kernel, int bytes, int dev)
{
    constexpr int SLOTS = 128;
    static std::atomic<const void *> fn[SLOTS];
    static std::atomic<unsigned long long> devs[SLOTS];
    if (dev >= 0 && dev < 64) {
        for (int i = 0; i < SLOTS; ++i) {
            const void *f = fn[i].load(std::memory_order_acquire);
            if (f == nullptr) {
                const void *expected = nullptr;
                if (fn[i].compare_exchange_strong(expected, kernel, std::memory_order_acq_rel)) f = kernel;
                else f = expected;
            }
            if (f != kernel) continue;
            if ((devs[i].load(std::memory_order_acquire) >> dev) & 1ull) return cudaSuccess;
            const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e == cudaSuccess) devs[i].fetch_or(1ull << dev, std::memory_order_release);
            return e;
        }
    }
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x)
{
    return __float2bfloat16_rn(x);
}

// Element idx of a pseudo-value array U, which the caller keeps in fp32 or (u_half) in fp16.
__device__ __forceinline__ float load_u(const void *U, size_t idx, int u_half)
{
    return u_half ? __half2float(static_cast<const __half *>(U)[idx]) : static_cast<const float *>(U)[idx];
}
__device__ __forceinline__ void store_u(void *U, size_t idx, float x, int u_half)
{
    if (u_half) static_cast<__half *>(U)[idx] = __float2half_rn(x);
    else static_cast<float *>(U)[idx] = x;
}

// Two packed bf16 (low = first element) -> two floats.  bf16 -> fp32 is a 16-bit shift.
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&p);
}

// 128 consecutive elements (16-byte aligned) widened into registers with 128-bit loads.
__device__ __forceinline__ void load_row128(const float *__restrict__ p, float (&s)[128])
{
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float4 x = reinterpret_cast<const float4 *>(p)[i];
        s[4 * i] = x.x, s[4 * i + 1] = x.y, s[4 * i + 2] = x.z, s[4 * i + 3] = x.w;
    }
}
__device__ __forceinline__ void load_row128(const __nv_bfloat16 *__restrict__ p, float (&s)[128])
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint4 x = reinterpret_cast<const uint4 *>(p)[i];
        s[8 * i] = bf16lo(x.x), s[8 * i + 1] = bf16hi(x.x);
        s[8 * i + 2] = bf16lo(x.y), s[8 * i + 3] = bf16hi(x.y);
        s[8 * i + 4] = bf16lo(x.z), s[8 * i + 5] = bf16hi(x.z);
        s[8 * i + 6] = bf16lo(x.w), s[8 * i + 7] = bf16hi(x.w);
    }
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// state slot of sequence b (block-pool addressing), or -1 when the index is out of range
__device__ __forceinline__ int state_slot(const int32_t *state_index, int n_states, int b)
{
    if (!state_index) return b;
    const int s = state_index[b];
    return (s >= 0 && s < n_states) ? s : -1;
}

__device__ __forceinline__ int nth_set_bit(unsigned long long m, int p)
{
#pragma unroll 1
    for (int q = 0; q < p; ++q) m &= m - 1;  // (rolled: the callers' code has to stay small)
    return __ffsll((long long)m) - 1;
}

__device__ __forceinline__ void widen8(const uint4 &x, float (&f)[8])
{
    f[0] = bf16lo(x.x), f[1] = bf16hi(x.x), f[2] = bf16lo(x.y), f[3] = bf16hi(x.y);
    f[4] = bf16lo(x.z), f[5] = bf16hi(x.z), f[6] = bf16lo(x.w), f[7] = bf16hi(x.w);
}

// stores that are predicated instead of branched around (keeps the epilogue one straight line)
__device__ __forceinline__ void st_global_if(float *p, float v, bool on)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t@q st.global.f32 [%0], %1;\n\t}" ::"l"(p), "f"(v),
                 "r"((int)on));
}
__device__ __forceinline__ void st_global_if(__nv_bfloat16 *p, float v, bool on)
{
    const unsigned short b = __bfloat16_as_ushort(__float2bfloat16_rn(v));
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t@q st.global.b16 [%0], %1;\n\t}" ::"l"(p), "h"(b),
                 "r"((int)on));
}

__device__ __forceinline__ void st_global_if(__half *p, float v, bool on)
{
    const unsigned short b = __half_as_ushort(__float2half_rn(v));
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t@q st.global.b16 [%0], %1;\n\t}" ::"l"(p), "h"(b),
                 "r"((int)on));
}

// Whether the packed range [lo, lo + n) of a sequence leaves the T packed nodes the caller declared
// (a stale or non-monotone node_offsets array): such a sequence is flagged and skipped before any of
// its rows is addressed.
__device__ __forceinline__ bool bad_offsets(int lo, int n, int T)
{
    return lo < 0 || n < 0 || (long long)lo + n > (long long)T;
}

// Status bits of sequence [lo, lo+n) of T packed nodes: range inside the packed arrays, node count in
// 1..max_nodes, parent[i] in -1..i-1.
// Called by every thread of a CTA with the same arguments; `scratch` is one shared int the
// caller zeroed before a barrier.  Returns the same value in every thread.
__device__ __forceinline__ int validate_sequence(const int32_t *__restrict__ parent, int lo, int n, int T,
                                                 int max_nodes, int *scratch)
{
    if (bad_offsets(lo, n, T)) return TREEWY_SEQ_BAD_OFFSETS;
    if (n < 1 || n > max_nodes) return TREEWY_SEQ_TOO_MANY_NODES;
    int bad = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int p = parent[lo + i];
        if (p < -1 || p >= i) bad = 1;
    }
    if (bad) atomicOr(scratch, TREEWY_SEQ_BAD_PARENT);
    __syncthreads();
    return *scratch;
}

}  // namespace treewy
