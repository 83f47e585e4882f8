// Host-side construction of TMA tensor maps for the KV pools (used by the tile and the streaming kernel).
// cuTensorMapEncodeTiled is fetched through the runtime's driver entry point, so nothing links against libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hat {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// A K or V pool as a 4-D tensor (column, slot, head, page) read in boxes of 64 columns x 16 slots (one page of one
// head, one 128-byte column half) with the 128-byte shared-memory swizzle.  Strides are in elements.
inline bool tma_encode_pool_map(CUtensorMap* map, bool bf16, const void* pool, int head_dim, int num_pages, int H,
                                int64_t stride_page, int64_t stride_token, int64_t stride_head) {
    EncodeTiledFn fn = tma_encode_fn();
    if (!fn || num_pages <= 0) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)head_dim, 16, (cuuint64_t)H, (cuuint64_t)num_pages};
    const cuuint64_t strides[3] = {(cuuint64_t)stride_token * 2, (cuuint64_t)stride_head * 2, (cuuint64_t)stride_page * 2};
    const cuuint32_t box[4] = {64, 16, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(pool),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The query rows [T][H][d] as a 3-D tensor (column, head, row) read in boxes of 64 columns x 128 rows of one head.
inline bool tma_encode_q_map(CUtensorMap* map, bool bf16, const void* q, int T, int H, int head_dim) {
    EncodeTiledFn fn = tma_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)H, (cuuint64_t)T};
    const cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)H * head_dim * 2};
    const cuuint32_t box[3] = {64, 1, 128};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(q), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A row-major 16-bit matrix [rows][cols] as a 2-D tensor (column, row) read in boxes of 64 columns x box_rows rows.
inline bool tma_encode_matrix_map(CUtensorMap* map, bool bf16, const void* base, int64_t rows, int64_t cols, int box_rows) {
    EncodeTiledFn fn = tma_encode_fn();
    if (!fn || rows <= 0 || cols <= 0) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace hat
