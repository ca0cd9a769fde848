// Expert-parallel sharding of the routed layer (the paper compares a tensor-parallel layout with expert-parallel ones,
// "TP8/EP1" against "TP4/EP4"): rank r holds the experts [e_begin, e_end) and finishes the tokens
// [r * tokens_per_rank, (r + 1) * tokens_per_rank).  Every rank routes and sorts all tokens (cheap, and identical
// everywhere); the rows of its own experts are one contiguous range of the sorted order, which the expert-FFN kernels
// take as they are (the offsets array shifted by e_begin).  What changes is where an output row goes: not into the
// rank's own y_perm but into the buffer of the rank that finishes the row's token, at row (token - first token) * k +
// slot - through peer memory, straight from the down projection's epilogue.  After a barrier every rank runs the
// slot-ordered combine on its own buffer: the same fp32 rows in the same order as on one GPU, hence the same bits.
#include "moe_common.cuh"

namespace moe {

// row_dst[p] for the sorted rows p of this rank's experts; slot = perm[p], token = slot / k
__global__ void __launch_bounds__(256) ep_row_table_kernel(const int* __restrict__ perm, const int* __restrict__ offsets, int k, int H,
                                                          int e_begin, int e_end, float* const* __restrict__ owner_y, int world,
                                                          int tokens_per_rank, float** __restrict__ row_dst) {
  pdl_wait();  // the order comes from the permute kernels before this one
  pdl_launch_dependents();
  const int p0 = offsets[e_begin], p1 = offsets[e_end];
  const int p = p0 + static_cast<int>(blockIdx.x * blockDim.x + threadIdx.x);
  if (p >= p1) return;
  const int slot = perm[p], token = slot / k, j = slot - token * k;
  int owner = token / tokens_per_rank;
  if (owner >= world) owner = world - 1;  // (cannot happen for tokens_per_rank = ceil(T / world))
  row_dst[p] = owner_y[owner] + (static_cast<size_t>(token - owner * tokens_per_rank) * k + j) * static_cast<size_t>(H);
}

int launch_ep_row_table(const int* perm, const int* offsets, int k, int H, int e_begin, int e_end, float* const* owner_y, int world,
                        int tokens_per_rank, float** row_dst, cudaStream_t st, int max_rows) {
  if (max_rows <= 0) return MOE_OK;
  if (launch_pdl(ep_row_table_kernel, dim3(static_cast<unsigned>((max_rows + 255) / 256)), dim3(256), 0, st, perm, offsets, k, H,
                 e_begin, e_end, owner_y, world, tokens_per_rank, row_dst) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel("ep_row_table", 1);
  return MOE_OK;
}

}  // namespace moe
