#include "tensormap.cuh"
#include <cstring>
#include <mutex>

namespace moa {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Encoded maps are kept in a small per-thread table keyed by everything that went into them (address, type, extents,
// strides, box, swizzle): a fused call needs eleven maps, and a step on the same buffers -- a training loop, a CUDA
// graph being re-recorded, a benchmark -- would otherwise encode the same eleven again (about a microsecond each: 56 us
// of host time per step against 39 us of kernels at B1 H32 n512).  A map describes memory, not its contents, so a
// cached one stays valid for as long as the caller's buffer keeps its address and shape.
struct MapKey {
    const void *base;
    uint64_t gdim[5], gstride[4];
    uint32_t box[5];
    uint32_t rank, dt, sw;
    bool operator==(const MapKey &o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    bool used;
};
constexpr int kMapSlots = 256;

uint64_t hash_key(const MapKey &k)
{
    const uint64_t *w = reinterpret_cast<const uint64_t *>(&k);
    uint64_t h = 0x9E3779B97F4A7C15ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; ++i) h = (h ^ w[i]) * 0xBF58476D1CE4E5B9ull + (h >> 29);
    return h;
}

EncodeTiledFn encode_fn();

// cuTensorMapEncodeTiled through the table
bool encode_cached(CUtensorMap *map, CUtensorMapDataType dt, uint32_t rank, const void *base, const cuuint64_t *gdim,
                   const cuuint64_t *gstride, const cuuint32_t *box, CUtensorMapSwizzle sw)
{
    static_assert(sizeof(MapKey) % 8 == 0, "hashed as 64-bit words");
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    thread_local MapSlot table[kMapSlots];
    MapKey k;
    memset(&k, 0, sizeof(k));
    k.base = base;
    for (uint32_t i = 0; i < rank; ++i) { k.gdim[i] = gdim[i]; k.box[i] = box[i]; }
    for (uint32_t i = 0; i + 1 < rank; ++i) k.gstride[i] = gstride[i];
    k.rank = rank; k.dt = (uint32_t)dt; k.sw = (uint32_t)sw;
    MapSlot &slot = table[hash_key(k) % kMapSlots];
    if (slot.used && slot.key == k) {
        *map = slot.map;
        return true;
    }
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (fn(map, dt, rank, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    slot.key = k;
    slot.map = *map;
    slot.used = true;
    return true;
}

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
    cuuint64_t gdim[3] = {cols, rows, heads};
    cuuint64_t gstride[2] = {cols * (uint64_t)elem_bytes, rows * cols * (uint64_t)elem_bytes};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return encode_cached(map, dt, 3, base, gdim, gstride, box, sw);
}

bool make_tensor_map_4d(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                        uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, bool bnhd,
                        uint32_t box_rows, uint32_t box_cols)
{
    const uint64_t eb = (uint64_t)elem_bytes;
    const uint64_t row_stride = (bnhd ? heads * cols : cols) * eb;
    const uint64_t head_stride = (bnhd ? cols : rows * cols) * eb;
    const uint64_t batch_stride = heads * rows * cols * eb;
    cuuint64_t gdim[4] = {cols, rows, heads, batch};
    cuuint64_t gstride[3] = {row_stride, head_stride, batch_stride};
    cuuint32_t box[4] = {box_cols, box_rows, 1, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return encode_cached(map, dt, 4, base, gdim, gstride, box, sw);
}

bool make_tensor_map_4d_strided(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                                uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, long long row_stride,
                                long long head_stride, long long batch_stride, uint32_t box_rows, uint32_t box_cols)
{
    if (row_stride <= 0 || head_stride <= 0 || batch_stride <= 0) return false;
    const uint64_t eb = (uint64_t)elem_bytes;
    cuuint64_t gdim[4] = {cols, rows, heads, batch};
    cuuint64_t gstride[3] = {(uint64_t)row_stride * eb, (uint64_t)head_stride * eb, (uint64_t)batch_stride * eb};
    cuuint32_t box[4] = {box_cols, box_rows, 1, 1};
    const CUtensorMapSwizzle sw =
        (box_cols * (uint32_t)elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return encode_cached(map, dt, 4, base, gdim, gstride, box, sw);
}

bool make_tensor_map_blocked(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                             uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t nblk)
{
    if (cols % 64 != 0 || elem_bytes != 2) return false;
    const uint64_t eb = (uint64_t)elem_bytes;
    cuuint64_t gdim[3] = {64, rows, cols / 64};
    cuuint64_t gstride[2] = {cols * eb, 64 * eb};          // row stride, then the 128-byte step between column blocks
    cuuint32_t box[3] = {64, box_rows, nblk};
    return encode_cached(map, dt, 3, base, gdim, gstride, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

}  // namespace moa
