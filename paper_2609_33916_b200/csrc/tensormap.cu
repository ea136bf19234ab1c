#include "tensormap.cuh"
#include <mutex>

namespace moa {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}
}  // namespace

bool make_tensor_map_3d(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                        uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {cols, rows, heads};
    cuuint64_t gstride[2] = {cols * (uint64_t)elem_bytes, rows * cols * (uint64_t)elem_bytes};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return fn(map, dt, 3, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tensor_map_4d(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                        uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, bool bnhd,
                        uint32_t box_rows, uint32_t box_cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const uint64_t eb = (uint64_t)elem_bytes;
    const uint64_t row_stride = (bnhd ? heads * cols : cols) * eb;
    const uint64_t head_stride = (bnhd ? cols : rows * cols) * eb;
    const uint64_t batch_stride = heads * rows * cols * eb;
    cuuint64_t gdim[4] = {cols, rows, heads, batch};
    cuuint64_t gstride[3] = {row_stride, head_stride, batch_stride};
    cuuint32_t box[4] = {box_cols, box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return fn(map, dt, 4, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tensor_map_4d_strided(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                                uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, long long row_stride,
                                long long head_stride, long long batch_stride, uint32_t box_rows, uint32_t box_cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn || row_stride <= 0 || head_stride <= 0 || batch_stride <= 0) return false;
    const uint64_t eb = (uint64_t)elem_bytes;
    cuuint64_t gdim[4] = {cols, rows, heads, batch};
    cuuint64_t gstride[3] = {(uint64_t)row_stride * eb, (uint64_t)head_stride * eb, (uint64_t)batch_stride * eb};
    cuuint32_t box[4] = {box_cols, box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return fn(map, dt, 4, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tensor_map_blocked(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                             uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t nblk)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64 != 0 || elem_bytes != 2) return false;
    const uint64_t eb = (uint64_t)elem_bytes;
    cuuint64_t gdim[3] = {64, rows, cols / 64};
    cuuint64_t gstride[2] = {cols * eb, 64 * eb};          // row stride, then the 128-byte step between column blocks
    cuuint32_t box[3] = {64, box_rows, nblk};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, dt, 3, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace moa
