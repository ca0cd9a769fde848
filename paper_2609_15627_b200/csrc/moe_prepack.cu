// moe_prepack: one-time re-layout of the expert weights (see ExpertWeights in moe_common.cuh).  Same bytes, same
// 4.25 bits per weight; for shapes that do not take the tile-contiguous layout it is a plain copy.
#include "moe_common.cuh"

namespace moe {

namespace {
// src: [rows][row_bytes]; dst: tiles of [128 rows][tile_bytes], tile (row / 128, byte / tile_bytes), the tiles of one
// row block consecutive.  One thread moves 16 bytes.
__global__ void __launch_bounds__(256) retile_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, size_t rows,
                                                    int row_bytes, int tile_bytes) {
  const size_t chunks_per_row = static_cast<size_t>(row_bytes) / 16;
  const size_t n = rows * chunks_per_row;
  const int tiles_per_row = row_bytes / tile_bytes, chunks_per_tile_row = tile_bytes / 16;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t row = i / chunks_per_row;
    const int c = static_cast<int>(i % chunks_per_row);
    const int tile = c / chunks_per_tile_row, cc = c % chunks_per_tile_row;
    const size_t o = ((row >> 7) * tiles_per_row + tile) * (static_cast<size_t>(128) * tile_bytes) + (row & 127) * tile_bytes + cc * 16;
    *reinterpret_cast<uint4*>(dst + o) = __ldg(reinterpret_cast<const uint4*>(src + i * 16));
  }
}

int retile(const uint8_t* src, uint8_t* dst, size_t rows, int row_bytes, int tile_bytes, cudaStream_t st) {
  const size_t n = rows * (static_cast<size_t>(row_bytes) / 16);
  const unsigned grid = static_cast<unsigned>(n / 256 + 1 < 148 * 16 ? n / 256 + 1 : 148 * 16);
  retile_kernel<<<grid, 256, 0, st>>>(src, dst, rows, row_bytes, tile_bytes);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
}  // namespace

int launch_prepack(const uint8_t* w13, const uint8_t* s13, const uint8_t* w2, const uint8_t* s2, const moe_shape_t& s,
                   uint8_t* packed, cudaStream_t st) {
  const PackedLayout L = packed_layout(s);
  const size_t n = static_cast<size_t>(s.E) * s.H * s.I;
  if (!blocked_shape(s)) {
    if (cudaMemcpyAsync(packed + L.w13, w13, n, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(packed + L.s13, s13, n / 16, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(packed + L.w2, w2, n / 2, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(packed + L.s2, s2, n / 32, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return MOE_ERR_CUDA;
    note_kernel("prepack_copy", 0);
    return MOE_OK;
  }
  const size_t r13 = static_cast<size_t>(s.E) * 2 * s.I, r2 = static_cast<size_t>(s.E) * s.H;
  int rc;
  if ((rc = retile(w13, packed + L.w13, r13, s.H / 2, 128, st)) != MOE_OK) return rc;
  if ((rc = retile(s13, packed + L.s13, r13, s.H / 32, 16, st)) != MOE_OK) return rc;
  if ((rc = retile(w2, packed + L.w2, r2, s.I / 2, 128, st)) != MOE_OK) return rc;
  if ((rc = retile(s2, packed + L.s2, r2, s.I / 32, 16, st)) != MOE_OK) return rc;
  note_kernel("prepack_retile", 4);
  return MOE_OK;
}

}  // namespace moe
