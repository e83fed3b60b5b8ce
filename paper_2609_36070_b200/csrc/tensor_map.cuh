// Host-side construction of TMA tensor maps, shared by the launchers of all tcgen05 kernels.  cuTensorMapEncodeTiled is
// reached through the runtime's driver entry point, so the library does not link against libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mok {
namespace tmap {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2D row-major tensor [rows, cols] of `elem_bytes`-wide elements whose rows are `row_stride_bytes` apart; one box =
// [box_rows x box_cols] elements.  The base must be 16-byte aligned and the stride a multiple of 16 bytes (checked by
// the driver); out-of-range parts of a box are filled with zeros on loads and clipped on stores.
inline bool encode_2d(CUtensorMap* m, CUtensorMapDataType dtype, const void* ptr, uint64_t rows, uint64_t cols,
                      uint64_t row_stride_bytes, uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, dtype, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 [rows, cols], rows `row_stride_elems` elements apart (0 = cols): boxes of [box_rows x 64] with the 128-byte swizzle
inline bool bf16_sw128(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
                       uint64_t row_stride_elems = 0) {
    return encode_2d(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ptr, rows, cols, (row_stride_elems ? row_stride_elems : cols) * 2,
                     64, box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

}  // namespace tmap
}  // namespace mok
