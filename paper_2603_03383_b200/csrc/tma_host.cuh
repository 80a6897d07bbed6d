// Host side of the 2-D TMA loads: a tensor map over a row-major bf16 matrix whose box is 64 columns
// (one 128-byte swizzle span) by box_rows rows.  The driver entry point is looked up once.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace mtv {

typedef CUresult (*TmaEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                               const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static inline TmaEncodeFn tma_encode_fn() {
    static TmaEncodeFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TmaEncodeFn>(ptr);
    }
    return fn;
}
// [rows][H] bf16 row-major, box = 64 columns x box_rows rows, 128-byte swizzle
static inline bool tma_map_2d_bf16(CUtensorMap *map, const void *base, int rows, int H, int box_rows) {
    TmaEncodeFn fn = tma_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    const cuuint64_t str[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t ones[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, str, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace mtv
