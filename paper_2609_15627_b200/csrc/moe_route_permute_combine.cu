// Router top-k, route production (stable expert sort + row gather) and the fixed-order fp32 combine.
// All three are integer / bandwidth work: warp shuffles, shared-memory histograms, prefix scans and
// 16-byte vector copies.  Results are bit-defined (see include/moe_b200.h).
#include "moe_common.cuh"
#include "moe_route_device.cuh"

namespace moe {

// =================================================================================================
// moe_route
// =================================================================================================

// Exclusive scan of counts[0..E) into offsets[0..E], offsets[E] = total.  Whole block takes part.
__device__ void block_offsets_scan(const int* counts, int E, int* offsets, int* warp_tot /* smem [32] */) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  const int per = (E + blockDim.x - 1) / blockDim.x;
  const int base = tid * per;
  int sum = 0;
  for (int i = 0; i < per; ++i)
    if (base + i < E) sum += counts[base + i];
  int wtotal;
  const int excl = warp_excl_scan(sum, lane, &wtotal);
  if (lane == 0) warp_tot[wid] = wtotal;
  __syncthreads();
  if (wid == 0) {
    const int v = (lane < nw) ? warp_tot[lane] : 0;
    int tot;
    const int ex = warp_excl_scan(v, lane, &tot);
    __syncwarp();
    warp_tot[lane] = ex;
    if (lane == 0) offsets[E] = tot;
  }
  __syncthreads();
  int run = warp_tot[wid] + excl;
  for (int i = 0; i < per; ++i) {
    if (base + i < E) {
      offsets[base + i] = run;
      run += counts[base + i];
    }
  }
}

// single_block != 0: one CTA handles every token and builds the histogram in shared memory.
// Otherwise the histogram is accumulated in g_counts[0..E) (zeroed before the launch) and the last
// CTA to finish (ticket in g_counts[E]) scans it.
__global__ void __launch_bounds__(1024) route_kernel(const float* __restrict__ logits, int T, int E, int k,
                                                     int* __restrict__ ids, float* __restrict__ w,
                                                     int* __restrict__ offsets, int* g_counts, int single_block) {
  extern __shared__ float sm_f[];
  const int nw = blockDim.x >> 5;
  float* rows = sm_f;                                   // [nw][E]
  int* s_counts = reinterpret_cast<int*>(sm_f + nw * E);  // [E]
  int* s_misc = s_counts + E;                           // [32] + flag
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  // Programmatic dependent launch on both sides: moe_permute may start and waits before it reads; this kernel may
  // itself have started while the kernel before it (the previous layer call's moe_combine, which still reads the
  // routing weights this kernel is about to overwrite) is running, so it reads only its input before it waits and
  // writes nothing to global memory until then.
  pdl_launch_dependents();
  bool waited = false;
  if (single_block) {
    for (int e = tid; e < E; e += blockDim.x) s_counts[e] = 0;
    __syncthreads();
  }
  float* row = rows + wid * E;
  const int t0 = blockIdx.x * nw + wid;
  const int tstride = gridDim.x * nw;
  for (int t = t0; t < T; t += tstride) {
    for (int e = lane; e < E; e += 32) row[e] = logits[static_cast<size_t>(t) * E + e];
    __syncwarp();
    int my_id;
    float my_v;
    warp_topk(row, E, k, lane, &my_id, &my_v);
    const float wt = warp_softmax_selected(my_v, k, lane);
    if (!waited) {
      pdl_wait();
      waited = true;
    }
    if (lane < k) {
      ids[static_cast<size_t>(t) * k + lane] = my_id;
      w[static_cast<size_t>(t) * k + lane] = wt;
      if (my_id >= 0) atomicAdd(single_block ? &s_counts[my_id] : &g_counts[my_id], 1);
    }
    __syncwarp();
  }
  if (!waited) pdl_wait();  // warps without a token
  if (single_block) {
    __syncthreads();
    block_offsets_scan(s_counts, E, offsets, s_misc);
    return;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_misc[32] = (atomicAdd(&g_counts[E], 1) == static_cast<int>(gridDim.x) - 1);
  __syncthreads();
  if (s_misc[32]) {
    __threadfence();
    for (int e = tid; e < E; e += blockDim.x) s_counts[e] = __ldcg(&g_counts[e]);
    __syncthreads();
    block_offsets_scan(s_counts, E, offsets, s_misc);
  }
}

int launch_route(const float* logits, int T, int E, int k, int* ids, float* w, int* offsets, int* counters,
                 cudaStream_t st) {
  const bool single = T <= 128;
  const int nw = single ? 32 : 8;
  const size_t smem = (static_cast<size_t>(nw) * E + E + 40) * 4;
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [] {
        return cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) == cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  int launches = 1;
  if (single) {
    if (launch_pdl(route_kernel, dim3(1), dim3(nw * 32), smem, st, logits, T, E, k, ids, w, offsets, counters, 1) != cudaSuccess)
      return MOE_ERR_CUDA;
    note_kernel("route_topk_single_cta", launches);
  } else {
    if (cudaMemsetAsync(counters, 0, (static_cast<size_t>(E) + 1) * 4, st) != cudaSuccess) return MOE_ERR_CUDA;
    const int grid = (T + nw - 1) / nw;
    route_kernel<<<grid, nw * 32, smem, st>>>(logits, T, E, k, ids, w, offsets, counters, 0);
    note_kernel("route_topk_multi_cta", launches);
  }
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// =================================================================================================
// moe_permute
// =================================================================================================

MOE_DEVINL void warp_copy_row(const __nv_bfloat16* src, __nv_bfloat16* dst, int H, int lane) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  const int n = H / 8;
  // eight loads in flight per lane: a row is a few KB and one warp moves it, so latency is what counts
  for (int i0 = lane; i0 < n; i0 += 32 * 8) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i0 + 32 * u < n) v[u] = __ldg(&s4[i0 + 32 * u]);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i0 + 32 * u < n) d4[i0 + 32 * u] = v[u];
  }
}

// Small S: one warp per slot.  Rank of slot s inside its expert = number of earlier slots with the
// same expert (counted directly), so the sort is stable by construction.
__global__ void __launch_bounds__(256) permute_small_kernel(const __nv_bfloat16* __restrict__ x,
                                                            const int* __restrict__ ids,
                                                            const int* __restrict__ offsets, int S, int H, int k,
                                                            __nv_bfloat16* __restrict__ x_perm,
                                                            int* __restrict__ perm, int* __restrict__ inv_perm) {
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  pdl_wait();                // the router's ids and offsets are complete
  pdl_launch_dependents();   // the expert FFN may set up and start its weight stream
  if (s >= S) return;
  const int e = ids[s];
  int c = 0;
  for (int q = lane; q < s; q += 32) c += (ids[q] == e);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
  const int p = offsets[e] + c;
  if (lane == 0) {
    perm[p] = s;
    inv_perm[s] = p;
  }
  warp_copy_row(x + static_cast<size_t>(s / k) * H, x_perm + static_cast<size_t>(p) * H, H, lane);
}

// Large S, pass 1: per-chunk histogram.
__global__ void __launch_bounds__(256) permute_count_kernel(const int* __restrict__ ids, int S, int E,
                                                            int* __restrict__ block_counts) {
  extern __shared__ int s_hist[];
  for (int e = threadIdx.x; e < E; e += blockDim.x) s_hist[e] = 0;
  __syncthreads();
  const int base = blockIdx.x * kPermuteChunk;
  for (int i = threadIdx.x; i < kPermuteChunk; i += blockDim.x) {
    const int s = base + i;
    if (s < S) atomicAdd(&s_hist[ids[s]], 1);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) block_counts[static_cast<size_t>(blockIdx.x) * E + e] = s_hist[e];
}

// Large S, pass 2: one warp per expert turns the per-chunk counts into per-chunk start positions.
__global__ void __launch_bounds__(256) permute_scan_kernel(const int* __restrict__ offsets, int E, int nblk,
                                                           int* __restrict__ block_counts) {
  const int lane = threadIdx.x & 31;
  const int e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (e >= E) return;
  int running = offsets[e];
  for (int b0 = 0; b0 < nblk; b0 += 32) {
    const int b = b0 + lane;
    const int v = (b < nblk) ? block_counts[static_cast<size_t>(b) * E + e] : 0;
    int tot;
    const int ex = warp_excl_scan(v, lane, &tot);
    if (b < nblk) block_counts[static_cast<size_t>(b) * E + e] = running + ex;
    running += tot;
  }
}

// Large S, pass 3: stable ranks inside a chunk.  Each warp owns 128 consecutive slots; warps are
// ordered through a per-warp count table, lanes through a match mask.
__global__ void __launch_bounds__(256) permute_scatter_kernel(const int* __restrict__ ids, int S, int E,
                                                              const int* __restrict__ block_base,
                                                              int* __restrict__ perm, int* __restrict__ inv_perm) {
  extern __shared__ int s_w[];  // [8][E]
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  constexpr int kWarps = 8, kPerWarp = kPermuteChunk / kWarps;
  for (int i = tid; i < kWarps * E; i += blockDim.x) s_w[i] = 0;
  __syncthreads();
  int* mine = s_w + wid * E;
  const int base = blockIdx.x * kPermuteChunk + wid * kPerWarp;
  const unsigned lt = (1u << lane) - 1u;
  for (int it = 0; it < kPerWarp / 32; ++it) {
    const int s = base + it * 32 + lane;
    const int e = (s < S) ? ids[s] : E;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (e < E && (peers & lt) == 0u) mine[e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    int run = block_base[static_cast<size_t>(blockIdx.x) * E + e];
    for (int w = 0; w < kWarps; ++w) {
      const int c = s_w[w * E + e];
      s_w[w * E + e] = run;
      run += c;
    }
  }
  __syncthreads();
  for (int it = 0; it < kPerWarp / 32; ++it) {
    const int s = base + it * 32 + lane;
    const int e = (s < S) ? ids[s] : E;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (e < E) {
      const int p = mine[e] + __popc(peers & lt);
      perm[p] = s;
      inv_perm[s] = p;
    }
    __syncwarp();
    if (e < E && (peers & lt) == 0u) mine[e] += __popc(peers);
    __syncwarp();
  }
}

// Large S, pass 4: gather rows, one warp per sorted row.
// range: null, or two device words {first sorted row, row after the last} - only those rows are copied (a rank of an
// expert-parallel job needs the rows of its own experts only)
__global__ void __launch_bounds__(256) permute_gather_kernel(const __nv_bfloat16* __restrict__ x,
                                                             const int* __restrict__ perm, int S, int H, int k,
                                                             __nv_bfloat16* __restrict__ x_perm, const int* __restrict__ range_lo,
                                                             const int* __restrict__ range_hi) {
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int p_lo = range_lo != nullptr ? *range_lo : 0, p_hi = range_hi != nullptr ? *range_hi : S;
  for (int p = p_lo + blockIdx.x * wpb + (threadIdx.x >> 5); p < p_hi; p += gridDim.x * wpb) {
    const int s = perm[p];
    warp_copy_row(x + static_cast<size_t>(s / k) * H, x_perm + static_cast<size_t>(p) * H, H, lane);
  }
}

int launch_permute(const __nv_bfloat16* x, const int* ids, const int* offsets, const moe_shape_t& sh,
                   __nv_bfloat16* x_perm, int* perm, int* inv_perm, int* block_counts, cudaStream_t st, const int* range_lo,
                   const int* range_hi) {
  const int S = sh.T * sh.k;
  if (S <= 4096) {
    if (launch_pdl(permute_small_kernel, dim3((S + 7) / 8), dim3(256), 0, st, x, ids, offsets, S, sh.H, sh.k, x_perm, perm,
                   inv_perm) != cudaSuccess)
      return MOE_ERR_CUDA;
    note_kernel("permute_rank_by_count", 1);
  } else {
    const int nblk = (S + kPermuteChunk - 1) / kPermuteChunk;
    permute_count_kernel<<<nblk, 256, sh.E * 4, st>>>(ids, S, sh.E, block_counts);
    permute_scan_kernel<<<(sh.E + 7) / 8, 256, 0, st>>>(offsets, sh.E, nblk, block_counts);
    permute_scatter_kernel<<<nblk, 256, 8 * sh.E * 4, st>>>(ids, S, sh.E, block_counts, perm, inv_perm);
    const int grid = min((S + 7) / 8, sm_count() * 16);
    permute_gather_kernel<<<grid, 256, 0, st>>>(x, perm, S, sh.H, sh.k, x_perm, range_lo, range_hi);
    note_kernel("permute_chunked_scan", 4);
  }
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// =================================================================================================
// moe_combine
// =================================================================================================

// One thread per (token, 8 consecutive columns): k fused multiply-adds per column in slot order.
__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ y, const int* __restrict__ inv_perm,
                                                      const float* __restrict__ w, int T, int H, int k,
                                                      __nv_bfloat16* __restrict__ out) {
  const int groups = H / 8;
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  pdl_wait();                // the per-slot rows of the expert FFN are complete
  pdl_launch_dependents();   // the next call on the stream (the next layer call's router) may start its set-up
  if (idx >= static_cast<size_t>(T) * groups) return;
  const int t = static_cast<int>(idx / groups);
  const int c = static_cast<int>(idx % groups) * 8;
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
  // slots in groups of four: the four row indices, then the eight row loads, are in flight together; the
  // multiply-adds stay in slot order
  for (int j0 = 0; j0 < k; j0 += 4) {
    int p[4];
    float wj[4];
    float4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (j0 + u < k) {
        p[u] = __ldg(&inv_perm[static_cast<size_t>(t) * k + j0 + u]);
        wj[u] = __ldg(&w[static_cast<size_t>(t) * k + j0 + u]);
      }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (j0 + u < k) {
        const float4* src = reinterpret_cast<const float4*>(y + static_cast<size_t>(p[u]) * H + c);
        a[u] = __ldg(src);
        b[u] = __ldg(src + 1);
      }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (j0 + u < k) {
        acc[0] = __fmaf_rn(wj[u], a[u].x, acc[0]);
        acc[1] = __fmaf_rn(wj[u], a[u].y, acc[1]);
        acc[2] = __fmaf_rn(wj[u], a[u].z, acc[2]);
        acc[3] = __fmaf_rn(wj[u], a[u].w, acc[3]);
        acc[4] = __fmaf_rn(wj[u], b[u].x, acc[4]);
        acc[5] = __fmaf_rn(wj[u], b[u].y, acc[5]);
        acc[6] = __fmaf_rn(wj[u], b[u].z, acc[6]);
        acc[7] = __fmaf_rn(wj[u], b[u].w, acc[7]);
      }
  }
  __nv_bfloat162 o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
  *reinterpret_cast<uint4*>(out + static_cast<size_t>(t) * H + c) = *reinterpret_cast<uint4*>(o);
}

int launch_combine(const float* y_perm, const int* inv_perm, const float* w, const moe_shape_t& sh,
                   __nv_bfloat16* out, cudaStream_t st) {
  const size_t n = static_cast<size_t>(sh.T) * (sh.H / 8);
  if (launch_pdl(combine_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, st, y_perm, inv_perm, w, sh.T,
                 sh.H, sh.k, out) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel("combine_slot_order_fma", 1);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// =================================================================================================
// moe_validate_scales
// =================================================================================================

__global__ void __launch_bounds__(256) validate_scales_kernel(const uint8_t* __restrict__ s, size_t n, int* bad) {
  int c = 0;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += static_cast<size_t>(gridDim.x) * blockDim.x)
    c += (s[i] > 128);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(bad, c);
}

int launch_validate_scales(const uint8_t* scales, size_t n, int* bad, cudaStream_t st) {
  if (cudaMemsetAsync(bad, 0, 4, st) != cudaSuccess) return MOE_ERR_CUDA;
  const int grid = static_cast<int>(min(static_cast<size_t>(sm_count()) * 8, (n + 255) / 256));
  validate_scales_kernel<<<grid > 0 ? grid : 1, 256, 0, st>>>(scales, n, bad);
  note_kernel("validate_scales", 1);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace moe
