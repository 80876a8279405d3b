// Host-side helpers for TMA tensor maps (driver entry point resolved through the runtime, so the
// library does not link libcuda).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace treewy {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn()
{
    // (looked up once per process: the entry point does not change, and the lookup is a microsecond
    // on every launch otherwise)
    static const EncodeTiledFn cached = [] {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<EncodeTiledFn>(fn);
    }();
    return cached;
}

// bf16 matrix [rows, cols] with `row_bytes` between rows; box = box_cols x box_rows
inline bool tma_make_map_bf16(EncodeTiledFn enc, CUtensorMap *m, const void *base, uint64_t cols,
                              uint64_t rows, uint64_t row_bytes, uint32_t box_cols, uint32_t box_rows,
                              CUtensorMapSwizzle sw)
{
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The four maps verify uses: S0 tiles, q rows, k rows (128-byte swizzle, 64-column boxes) and v rows.
struct VerifyMaps {
    CUtensorMap S0, Q, K, V;
};
inline bool make_verify_maps(VerifyMaps *m, const void *S0, const void *q, const void *k, const void *v,
                             long long n_items, int T, int H_v, int H_qk, int box_rows)
{
    EncodeTiledFn enc = tma_encode_fn();
    if (!enc) return false;
    const uint64_t D = 128;
    bool ok = tma_make_map_bf16(enc, &m->S0, S0, D, (uint64_t)n_items * D, D * 2, 64, 128,
                                CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && tma_make_map_bf16(enc, &m->Q, q, (uint64_t)H_qk * D, T, (uint64_t)H_qk * D * 2, 64, box_rows,
                                 CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && tma_make_map_bf16(enc, &m->K, k, (uint64_t)H_qk * D, T, (uint64_t)H_qk * D * 2, 64, box_rows,
                                 CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && tma_make_map_bf16(enc, &m->V, v, (uint64_t)H_v * D, T, (uint64_t)H_v * D * 2, 128, box_rows,
                                 CU_TENSOR_MAP_SWIZZLE_NONE);
    return ok;
}

}  // namespace treewy
