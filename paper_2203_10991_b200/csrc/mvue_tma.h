// Host-side helper: TMA tensor maps through the driver entry point (no link-time libcuda dependency).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <cstdint>
#include <mutex>

namespace mvue {

inline PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    });
    return fn;
}

// Row-major matrix of `outer` rows x `inner` elements, row pitch in bytes; box = box_inner x box_outer elements.
inline bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                        uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle) {
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {pitch_bytes};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, dtype, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A row-major bf16 matrix [rows x cols] (row pitch in bytes, rows a multiple of 16) seen as the 4-D tensor
// (col, k2, strip, k8) with row = 16 strip + 2 k8 + k2, box = 64 columns x 2 x `box_strips` x 8 with the 128-byte
// swizzle.  In shared memory the box is lines of 128 bytes, line = 2 box_strips k8 + 2 strip + k2: the eight lines
// {k8 fixed, strip s..s+3, k2 0..1} that one transposing 8x8 matrix load gathers sit in eight different swizzle
// phases, so the load has no bank conflict.
inline bool make_map_strips(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                            uint32_t box_strips) {
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[4] = {cols, 2, rows / 16, 8};
    const cuuint64_t strides[3] = {pitch_bytes, 16 * pitch_bytes, 2 * pitch_bytes};
    const cuuint32_t box[4] = {64, 2, box_strips, 8};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix (rows a multiple of 32) seen as the 5-D tensor (col, k2, pair, h, k8) with
// row = 32 pair + 16 h + 2 k8 + k2, box = 64 columns x 2 x 4 x 2 x 8 (128 rows) with the 128-byte swizzle.  In shared
// memory the box is lines of 128 bytes, line = 16 k8 + 8 h + 2 pair + k2: the eight lines {k8, h fixed, pair 0..3, k2 0..1}
// that one transposing 8x8 matrix load gathers are consecutive, hence in eight different swizzle phases (no bank
// conflict), and they hand lane l rows 2 k8, 2 k8 + 1 of strip 2 (l % 4) + h: a lane that loads h = 0 and h = 1 owns two
// consecutive strips -- 32 consecutive rows -- of its column.
inline bool make_map_strip_pairs(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes) {
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[5] = {cols, 2, rows / 32, 2, 8};
    const cuuint64_t strides[4] = {pitch_bytes, 32 * pitch_bytes, 16 * pitch_bytes, 2 * pitch_bytes};
    const cuuint32_t box[5] = {64, 2, 4, 2, 8};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace mvue
