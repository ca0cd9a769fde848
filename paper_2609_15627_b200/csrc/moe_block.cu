// The steps either side of the routed path (paper, figure "Execution structure": router scores before the Top-k, the
// shared expert beside the routed experts, "add partials" after them):
//   router projection   logits[T,E] = x[T,H] * w_router[E,H]^T, bf16 operands, fp32 accumulation
//   join                out = bf16( slot-ordered fp32 sum of the routed experts + the shared expert's fp32 row )
// The shared expert itself is one more expert in the routed experts' weight format applied to every token: it runs
// through the expert-FFN kernels with E = 1 (x as its own sorted rows, offsets {0, T}).
//
// Router projection, two kernels:
//   * up to 16 tokens: one warp per expert streams that expert's row of w_router once (16-byte loads, the whole matrix
//     is read once by the grid) against the token rows held in shared memory; lanes keep fp32 partial sums over their
//     strided share of H, a shuffle tree adds them.  Bound by the 2 MB read of w_router, a few microseconds.
//   * more tokens: a tcgen05 GEMM, kind::f16 on bf16, tile = 128 tokens x 64 experts, accumulator in tensor memory,
//     operands by TMA (128-byte swizzle) through a 4-stage ring; warp 0 loads, warp 1 issues the MMAs, warps 2..5
//     read the accumulator and store fp32 rows.  The paper kept a vendor BLAS here after two custom routers lost to it
//     on its hardware; on this one the projection is 0.5 % of the layer's flops and the tile shape is picked for the
//     number of CTAs (T/128 x E/64), not for the tensor-core rate.
#include <cuda.h>

#include "moe_sm100_primitives.cuh"
#include "moe_tmap.cuh"

namespace moe {

namespace {

constexpr int kGemvMaxTok = 16;
constexpr int kGemvWarps = 8;

__global__ void __launch_bounds__(kGemvWarps * 32) router_gemv_kernel(const __nv_bfloat16* __restrict__ x,
                                                                      const __nv_bfloat16* __restrict__ wr, int T, int H,
                                                                      int E, float* __restrict__ logits) {
  extern __shared__ __align__(16) unsigned char smem_x[];  // [T][H] bf16
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();  // x may be the output of the kernel before this one
  const int n16 = T * H / 8;
  for (int i = tid; i < n16; i += blockDim.x) reinterpret_cast<uint4*>(smem_x)[i] = __ldg(reinterpret_cast<const uint4*>(x) + i);
  __syncthreads();
  const int e = blockIdx.x * kGemvWarps + wid;
  if (e >= E) return;
  float acc[kGemvMaxTok];
#pragma unroll
  for (int t = 0; t < kGemvMaxTok; ++t) acc[t] = 0.0f;
  const uint4* wrow = reinterpret_cast<const uint4*>(wr + static_cast<size_t>(e) * H);
  for (int c0 = lane; c0 < H / 8; c0 += 32 * 4) {  // four 16-byte loads in flight per lane
    uint4 wv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (c0 + 32 * u < H / 8) wv[u] = __ldg(wrow + c0 + 32 * u);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + 32 * u;
      if (c < H / 8) {
        const uint32_t ww[4] = {wv[u].x, wv[u].y, wv[u].z, wv[u].w};
#pragma unroll
        for (int t = 0; t < kGemvMaxTok; ++t) {
          if (t < T) {
            const uint4 xv = *reinterpret_cast<const uint4*>(smem_x + (static_cast<size_t>(t) * H + c * 8) * 2);
            const uint32_t xx[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              acc[t] = fmaf(__uint_as_float(ww[i] << 16), __uint_as_float(xx[i] << 16), acc[t]);
              acc[t] = fmaf(__uint_as_float(ww[i] & 0xFFFF0000u), __uint_as_float(xx[i] & 0xFFFF0000u), acc[t]);
            }
          }
        }
      }
    }
  }
#pragma unroll
  for (int t = 0; t < kGemvMaxTok; ++t) {
    if (t < T) {
      float v = acc[t];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
      if (lane == 0) logits[static_cast<size_t>(t) * E + e] = v;
    }
  }
}

// ---- tcgen05 GEMM: tile of 128 tokens x 64 experts ----
constexpr int kRM = 128, kRN = 64, kRK = 64;  // K per stage: one 128-byte row of bf16
constexpr int kRStages = 4;
constexpr int kRABytes = kRM * kRK * 2, kRBBytes = kRN * kRK * 2;
constexpr int kRThreads = 6 * 32;

__global__ void __launch_bounds__(kRThreads, 1)
router_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, int T, int H, int E,
                   float* __restrict__ logits, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sA = smem;
  unsigned char* sB = smem + kRStages * kRABytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sB + kRStages * kRBBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kRStages;
  uint64_t* acc_full = empty + kRStages;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_full + 1);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int t0 = blockIdx.x * kRM, e0 = blockIdx.y * kRN;
  const int n_kb = H / kRK;
  if (tid == 0) {
    for (int s = 0; s < kRStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
  }
  if (wid == 1) tmem_alloc(tmem_holder, 64);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  if (wid == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int kb = 0; kb < n_kb; ++kb) {
        mbar_wait(&empty[s], ph ^ 1u, status);
        mbar_expect_tx(&full[s], kRABytes + kRBBytes);
        tma_load_2d(sA + s * kRABytes, &tmap_x, kb * kRK, t0, &full[s]);   // rows past T arrive as zeros
        tma_load_2d(sB + s * kRBBytes, &tmap_w, kb * kRK, e0, &full[s]);   // rows past E likewise
        if (++s == kRStages) { s = 0; ph ^= 1u; }
      }
    }
  } else if (wid == 1) {
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      const uint32_t idesc = umma_idesc_bf16(kRM, kRN);
      for (int kb = 0; kb < n_kb; ++kb) {
        mbar_wait(&full[s], ph, status);
        tc_fence_after_sync();
        const uint32_t a_addr = smem_u32(sA + s * kRABytes), b_addr = smem_u32(sB + s * kRBBytes);
#pragma unroll
        for (int k4 = 0; k4 < kRK / 16; ++k4)
          umma_bf16(tmem_base, umma_desc_k_sw128(a_addr + k4 * 32), umma_desc_k_sw128(b_addr + k4 * 32), idesc, (kb | k4) != 0 ? 1u : 0u);
        umma_commit(&empty[s]);
        if (++s == kRStages) { s = 0; ph ^= 1u; }
      }
      umma_commit(acc_full);
    }
  } else {
    const int q = wid & 3;  // tensor-memory lane quadrant: token row t0 + 32 q + lane
    mbar_wait(acc_full, 0u, status);
    __syncwarp();
    tc_fence_after_sync();
    const int t = t0 + 32 * q + lane;
#pragma unroll 1
    for (int c0 = 0; c0 < kRN; c0 += 32) {
      uint32_t v[32];
      tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c0), v);
      tmem_ld_wait();
      if (t < T) {
        float* dst = logits + static_cast<size_t>(t) * E + e0 + c0;
        if (e0 + c0 + 32 <= E && (E & 3) == 0) {
#pragma unroll
          for (int i = 0; i < 32; i += 4)
            *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]), __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (e0 + c0 + i < E) dst[i] = __uint_as_float(v[i]);
        }
      }
    }
    tc_fence_before_sync();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 64);
  }
}

// ---- join: the slot-ordered fp32 sum of the routed experts (moe_combine's recurrence) + the shared expert's row ----
__global__ void __launch_bounds__(256) combine_shared_kernel(const float* __restrict__ y, const int* __restrict__ inv_perm,
                                                             const float* __restrict__ w, const float* __restrict__ y_shared,
                                                             int T, int H, int k, __nv_bfloat16* __restrict__ out) {
  const int groups = H / 8;
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  if (idx >= static_cast<size_t>(T) * groups) return;
  const int t = static_cast<int>(idx / groups);
  const int c = static_cast<int>(idx % groups) * 8;
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
  const float4* sh = reinterpret_cast<const float4*>(y_shared + static_cast<size_t>(t) * H + c);
  const float4 s0 = __ldg(sh), s1 = __ldg(sh + 1);
  for (int j0 = 0; j0 < k; j0 += 4) {  // four slots' rows in flight; the multiply-adds stay in slot order
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
  const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
  __nv_bfloat162 o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = __floats2bfloat162_rn(__fadd_rn(acc[2 * i], sv[2 * i]), __fadd_rn(acc[2 * i + 1], sv[2 * i + 1]));
  *reinterpret_cast<uint4*>(out + static_cast<size_t>(t) * H + c) = *reinterpret_cast<uint4*>(o);
}

__global__ void shared_offsets_kernel(int* offsets, int T) {
  // waits BEFORE it releases its dependent: moe_route, launched next, reads the logits before its own wait, so the
  // router projection two launches back must be complete by the time moe_route may start
  pdl_wait();
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    offsets[0] = 0;
    offsets[1] = T;
  }
}

}  // namespace

int launch_router_logits(const __nv_bfloat16* x, const __nv_bfloat16* w_router, int T, int H, int E, float* logits, int* status,
                         cudaStream_t st) {
  if (T <= kGemvMaxTok && static_cast<size_t>(T) * H * 2 <= 160 * 1024) {
    const size_t smem = static_cast<size_t>(T) * H * 2;
    static PerDeviceFlag flag;
    if (!once_per_device(flag, [] {
          return cudaFuncSetAttribute(router_gemv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024) == cudaSuccess;
        }))
      return MOE_ERR_CUDA;
    if (launch_pdl(router_gemv_kernel, dim3((E + kGemvWarps - 1) / kGemvWarps), dim3(kGemvWarps * 32), smem, st, x, w_router, T, H, E,
                   logits) != cudaSuccess)
      return MOE_ERR_CUDA;
    note_kernel("router_gemv_warp_per_expert", 1);
    return MOE_OK;
  }
  CUtensorMap tm_x, tm_w;
  if (!bf16_map_2d(&tm_x, x, H, T, kRK, kRM) || !bf16_map_2d(&tm_w, w_router, H, E, kRK, kRN)) return MOE_ERR_CUDA;
  const size_t smem = kRStages * (kRABytes + kRBBytes) + 256 + 1024;
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [smem] {
        return cudaFuncSetAttribute(router_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) == cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  router_gemm_kernel<<<dim3((T + kRM - 1) / kRM, (E + kRN - 1) / kRN), kRThreads, smem, st>>>(tm_x, tm_w, T, H, E, logits, status);
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  note_kernel("router_gemm_tcgen05_128x64", 1);
  return MOE_OK;
}

int launch_combine_shared(const float* y_perm, const int* inv_perm, const float* w, const float* y_shared, const moe_shape_t& sh,
                          __nv_bfloat16* out, cudaStream_t st) {
  const size_t n = static_cast<size_t>(sh.T) * (sh.H / 8);
  if (launch_pdl(combine_shared_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, st, y_perm, inv_perm, w, y_shared,
                 sh.T, sh.H, sh.k, out) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel("combine_slot_order_fma_plus_shared", 1);
  return MOE_OK;
}

int launch_shared_offsets(int* offsets2, int T, cudaStream_t st) {
  if (launch_pdl(shared_offsets_kernel, dim3(1), dim3(32), 0, st, offsets2, T) != cudaSuccess) return MOE_ERR_CUDA;
  note_kernel("shared_expert_offsets", 1);
  return MOE_OK;
}

}  // namespace moe
