// Host helper: builds CUtensorMap descriptors through the driver entry point (no link against libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ql {

// 2-D row-major int8 tensor [rows][cols] (cols innermost), box [box_rows][box_cols], 128-byte swizzle.
// cols must be a multiple of 16 and base 16-byte aligned.  Out-of-range box elements read as zero.
bool make_tensor_map_i8(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                        uint32_t box_cols);
// 2-D row-major int16 tensor, no swizzle.
bool make_tensor_map_i16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols);

}  // namespace ql
