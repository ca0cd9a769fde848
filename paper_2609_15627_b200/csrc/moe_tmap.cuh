// Tensor maps (TMA descriptors) of the expert weights, shared by the kernels that stream them with
// cp.async.bulk.tensor: a 128-byte-swizzled box of 128 rows x 128 bytes of packed codes and a box of 128 rows x 16
// scale bytes, over the checkpoint's row layout or over moe_prepack's tile-contiguous layout (see ExpertWeights).
#pragma once

#include <cuda.h>

#include "moe_common.cuh"

namespace moe {

bool weight_maps(const ExpertWeights& w, const moe_shape_t& sh, CUtensorMap* tm_w13, CUtensorMap* tm_s13, CUtensorMap* tm_w2,
                 CUtensorMap* tm_s2);

// E2M1 term rows of activations: byte tensor [rows][row_bytes], box of box_rows rows x 128 bytes, 128-byte swizzle
bool term_row_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_rows);

// bf16 matrix [rows][inner elements], box of box_rows rows x box_inner elements (128 bytes), 128-byte swizzle; rows past
// the end of the matrix read as zeros
bool bf16_map_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows);

}  // namespace moe
