// Host-side creation of TMA tensor maps for row-major bf16 matrices.
#include <cuda.h>

#include <cstring>

#include "common.cuh"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// A [rows, cols] row-major bf16 matrix viewed through boxes of [box_rows, 64]
// elements (128 bytes wide) stored with the 128-byte swizzle.  Rows past the
// end of the matrix read as zero.
bool make_tmap_bf16_rows(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || rows == 0 || cols % 64 != 0) return false;
    cuuint64_t gdim[2] = {cols, rows};
    cuuint64_t gstride[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estride[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box,
              estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Small cache so that steady-state calls on the same buffers re-encode nothing.
const CUtensorMap *TmapCache::get(const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    for (int i = 0; i < n; ++i)
        if (e[i].base == base && e[i].rows == rows && e[i].cols == cols && e[i].box_rows == box_rows)
            return &e[i].map;
    Entry &slot = e[next];
    if (!make_tmap_bf16_rows(&slot.map, base, rows, cols, box_rows)) return nullptr;
    slot.base = base; slot.rows = rows; slot.cols = cols; slot.box_rows = box_rows;
    const CUtensorMap *r = &slot.map;
    next = (next + 1) % kEntries;
    if (n < kEntries) ++n;
    return r;
}
