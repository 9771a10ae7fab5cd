// Host-side construction of TMA tensor maps.  cuTensorMapEncodeTiled is fetched from the driver at
// first use, so the library does not link libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace lrq_tma {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            p = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Row-major matrix [rows, cols] of `elem_bytes`-byte elements (1: uint8, 2: bf16, 4: fp32) with `ld` elements between
// rows; tiles of box_cols x box_rows elements; out-of-range elements read as zero.  The base pointer and the
// row pitch must be multiples of 16 bytes, box_cols * elem_bytes a multiple of 16 (and at most 128 with swizzle).
inline bool make_map_2d(CUtensorMap* tm, const void* ptr, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                        uint32_t box_cols, uint32_t box_rows, bool swizzle128) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
               const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 matrix [rows, cols] (cols a multiple of 64, `ld` elements between rows) seen as a 3-D tensor
// [rows][cols / 64][64], so that one copy brings `box_rows` whole rows into shared memory as consecutive 128-byte
// lines (64 elements each), 128-byte swizzled: the 16-byte chunk c of line L lands at chunk c ^ (L & 7).
inline bool make_map_rows_bf16(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc || cols % 64 || cols / 64 > 256 || box_rows < 1 || box_rows > 256) return false;
    const cuuint64_t dims[3] = {64, cols / 64, rows};
    const cuuint64_t strides[2] = {128, ld * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)(cols / 64), box_rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace lrq_tma
