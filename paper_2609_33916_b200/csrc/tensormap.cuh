// Host-side construction of TMA descriptors for [BH, n, d] tensors.
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

namespace moa {

// Tiled map over a contiguous [heads, rows, cols] tensor (cols fastest) with boxes of
// [1, box_rows, box_cols]; 128-byte swizzle when box_cols * elem_bytes == 128, none
// otherwise.  Out-of-range rows read as zero and are clipped on store/reduce.
// Returns false if the driver entry point is unavailable or the encode fails.
bool make_tensor_map_3d(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                        uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols);

// Tiled map over one of the caller's [B, heads, rows, cols] tensors in either memory layout
// (bnhd = false: [B,H,n,d] contiguous; true: [B,n,H,d] contiguous), as a 4-D tensor
// (cols, rows, heads, B) with boxes of [1, 1, box_rows, box_cols]; 128-byte swizzle when
// box_cols * elem_bytes == 128.  Rows past `rows` read as zero and are clipped on store.
bool make_tensor_map_4d(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                        uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, bool bnhd,
                        uint32_t box_rows, uint32_t box_cols);

// The same with explicit strides in ELEMENTS between rows, heads and batches (each a multiple of 16 bytes; the cols
// elements of a row are contiguous): any memory layout a caller's projection produces, e.g. the Q third of a packed
// [B, n, 3, H, d] array.
bool make_tensor_map_4d_strided(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                                uint64_t batch, uint64_t heads, uint64_t rows, uint64_t cols, long long row_stride,
                                long long head_stride, long long batch_stride, uint32_t box_rows, uint32_t box_cols);

// Map over a [rows, cols] array (cols fastest, cols a multiple of 64) seen as (64 columns, rows, cols/64 column
// blocks): one box of [nblk, box_rows, 64] lands in shared memory block by block -- nblk consecutive tiles of
// box_rows rows x 128 bytes, 128-byte swizzle -- which is the layout an MN-major UMMA operand wants, fetched by one
// copy instead of nblk.  Returns false when the encode is refused (the caller then uses one box per block).
bool make_tensor_map_blocked(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes,
                             uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t nblk);

}  // namespace moa
