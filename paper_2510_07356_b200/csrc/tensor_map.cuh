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

// The maps of recent (base address, shape) combinations, so that a caller that alternates between a few
// pools -- the layers of a model, one decode step after the other -- encodes each map once instead of
// on every call.  A map holds nothing but what the key holds, so a hit is exact.  Not thread-safe:
// it lives in a handle, and calls on one handle are ordered by the caller.
struct RowsMapCache {
    static constexpr int kEntries = 160;          // K and V pools of 64 layers, and some
    struct Entry {
        const void* base = nullptr;
        uint64_t rows = 0;
        uint32_t box_rows = 0, box_planes = 0, planes = 0;
        CUtensorMap map;
    };
    Entry e[kEntries];
    int used = 0, next = 0;

    const CUtensorMap* get(const void* base, uint64_t rows, uint32_t box_rows, uint32_t box_planes, uint32_t planes) {
        for (int i = 0; i < used; ++i)
            if (e[i].base == base && e[i].rows == rows && e[i].box_rows == box_rows && e[i].box_planes == box_planes &&
                e[i].planes == planes)
                return &e[i].map;
        Entry& x = e[next];
        if (!make_rows_map(&x.map, base, rows, box_rows, box_planes, planes)) { x.base = nullptr; return nullptr; }
        x.base = base; x.rows = rows; x.box_rows = box_rows; x.box_planes = box_planes; x.planes = planes;
        next = (next + 1) % kEntries;
        if (used < kEntries) ++used;
        return &x.map;
    }
};

}  // namespace concur
