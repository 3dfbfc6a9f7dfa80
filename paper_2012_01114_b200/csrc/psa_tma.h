// Host helper: builds 2-D TMA tensor maps for row-major bf16 / fp32 matrices.  The driver entry
// point is looked up through the runtime so that the library does not link against libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace psa {

// Tensor map over a row-major [rows x cols] matrix of 2-byte elements with `pitch_bytes` between
// rows; boxes are [box_rows x box_cols] with box_cols * 2 == 128 bytes, 128-byte swizzle.
// Returns false (and sets the error text) on failure.
bool make_tensor_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_bytes,
                          uint32_t box_rows, uint32_t box_cols);

// Tensor map over a [batch, n, heads, d] bf16 tensor (dense, d a multiple of 8): boxes are [1 x box_rows x 1 head x
// 64 elements]; elements beyond d and rows beyond n are out of bounds of the map (zero fill on load, dropped on store).
bool make_tensor_map_bf16_4d(CUtensorMap* map, const void* base, uint64_t batch, uint64_t n, uint64_t heads, uint64_t d,
                             uint32_t box_rows);

}  // namespace psa
