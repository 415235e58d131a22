// Host-side construction of TMA tensor maps.  The driver's encoder is reached through the
// runtime's entry-point query, so the library links against the CUDA runtime only.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lrd {

// 2-D bf16 tensor [rows x cols], row stride ld elements, box [box_rows x box_cols]; the swizzle
// span equals the box row (128, 64 or 32 bytes; none otherwise); zero fill outside the tensor.
// Returns false on failure.
bool make_tmap_2d_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld_elems,
                       uint32_t box_rows, uint32_t box_cols);

// 4-D bf16 NHWC tensor [B][H][W][C], box [1][box_h][box_w][box_c], 128-byte swizzle, zero fill.
bool make_tmap_nhwc_bf16(CUtensorMap* out, const void* base, uint64_t B, uint64_t H, uint64_t W, uint64_t C,
                         uint32_t box_h, uint32_t box_w, uint32_t box_c);

}  // namespace lrd
