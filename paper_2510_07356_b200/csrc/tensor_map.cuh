// Host-side construction of the TMA tensor maps the kernels use.  One shape serves every
// operand: a matrix of 128-element bf16 rows seen as {64 elements, rows, planes}, where a plane
// is one 64-element half of a row (element stride 2 B, plane stride 128 B, row stride
// planes x 128 B).  A box {64, box_rows, box_planes} lands in shared memory as
// [plane][row][128 B] with the 128-byte swizzle: conflict-free for ldmatrix and directly a
// K-major (or, read along the rows, MN-major) tcgen05 operand slab.
//
//   planes = 2                 q / out rows and head-major pools [page][head][slot][128]
//   planes = 2 x KV heads      token-major pools [page][slot][head][128]: row = token, plane 2g + half
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace concur {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
inline EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

inline bool make_rows_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows, uint32_t box_planes,
                          uint32_t planes = 2) {
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, rows, planes};
    const cuuint64_t strides[2] = {(cuuint64_t)planes * 128, 128};
    const cuuint32_t box[3] = {64, box_rows, box_planes};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace concur
