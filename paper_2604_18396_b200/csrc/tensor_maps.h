// Host helpers that encode the 2-D TMA tensor maps of weights, operand buffers and the KV pool (internal).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace river {

typedef CUresult (*TmapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline TmapEncodeFn tmap_encoder() {
    static TmapEncodeFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess) fn = (TmapEncodeFn)p;
    }
    return fn;
}
// row-major matrix [rows][inner] of 1- or 2-byte elements -> tiled map with a (box_rows x 128 byte) box and the
// 128-byte swizzle
inline bool make_map_2d(CUtensorMap *m, CUtensorMapDataType dt, int elem_bytes, const void *base, uint64_t inner,
                        uint64_t rows, uint32_t box_rows) {
    TmapEncodeFn fn = tmap_encoder();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {inner, rows};
    const cuuint64_t gstride[1] = {inner * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, dt, 2, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool make_map_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t rows, uint32_t box_rows) {
    return make_map_2d(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, inner, rows, box_rows);
}
// u8 code matrix [rows][inner_bytes]
inline bool make_map_codes(CUtensorMap *m, const void *base, uint64_t inner_bytes, uint64_t rows, uint32_t box_rows) {
    return make_map_2d(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base, inner_bytes, rows, box_rows);
}

}  // namespace river
