// Device routines shared by the kernels that feed the block-scaled FP4 tensor-core instruction (kind::mxf4): the MMA
// itself with its instruction descriptor, tensor-memory stores for scale factors, the split of a bf16 activation row
// into E2M1 term rows with per-32 block scales, and the bounded wait on a global counter.
#pragma once

#include <cuda_fp4.h>

#include "moe_sm100_primitives.cuh"

namespace moe {

constexpr int kTerms = 8;  // E2M1 terms per activation value: x = sum_t 2^(s_t) * q_t, residual below 2^-16 of the block's maximum

MOE_DEVINL void tmem_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
MOE_DEVINL void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem, E2M1] * B[smem, E2M1]^T, K = 64, two UE8M0 block scales per row held in tensor memory
MOE_DEVINL void umma_mxf4(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa, uint32_t sfb,
                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
      :
      : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
      : "memory");
}
// instruction descriptor: A and B E2M1, UE8M0 scales, M = 128, N = 256 (or n_cols); `half` (0 or 1) picks bytes 0,1 or
// 2,3 of the scale words
MOE_DEVINL uint32_t idesc_mxf4(uint32_t half, uint32_t n_cols = 256u) {
  return (1u << 7) | (1u << 10) | ((n_cols >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) | ((2u * half) << 29) | ((2u * half) << 4);
}

// Bounded wait until *p >= need (acquire at GPU scope); same give-up rules as mbar_wait
MOE_DEVINL void counter_wait_ge(const int* p, int need, int* status) {
  const long long t0 = clock64();
  int spins = 0;
  while (true) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    if (v >= need) return;
    const long long waited = clock64() - t0;
    if (waited > kWaitLimitCycles) {
      if (status != nullptr) atomicExch(status, static_cast<int>(MOE_ERR_TIMEOUT));
      return;
    }
    if (((++spins) & 63) == 0 && waited > 2000000 && status != nullptr && *reinterpret_cast<volatile int*>(status) != 0) return;
    __nanosleep(64);
  }
}
// orders this thread's generic-proxy accesses with its asynchronous-proxy (TMA) accesses, global memory included
MOE_DEVINL void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
MOE_DEVINL void prefetch_tmap(const void* tmap) { asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory"); }

MOE_DEVINL float pow2f(int e) { return __uint_as_float(static_cast<uint32_t>(e + 127) << 23); }  // e in [-126, 127]
// Block exponent of a term: the smallest s with amax <= 6 * 2^s (amax > 0), kept inside the UE8M0 range
MOE_DEVINL int term_exp(float amax) {
  const uint32_t u = __float_as_uint(amax);
  const int e = static_cast<int>((u >> 23) & 0xFFu) - 127;
  const int s = ((u & 0x7FFFFFu) <= 0x400000u) ? e - 2 : e - 1;  // 1.5 * 2^e = 6 * 2^(e-2)
  return max(-126, min(s, 126));
}
// Two values (already divided by the block scale) -> one byte of two E2M1 codes (a in the low nibble) and their
// decoded values.  (A version in plain float and integer instructions - step chosen by two compares, the multiple by
// the round-to-nearest-even of one float addition - gives the same codes and was slower: decode_c64 call +4 %.)
MOE_DEVINL uint32_t e2m1_pair(float a, float b, float* qa, float* qb) {
  const __nv_fp4x2_storage_t c = __nv_cvt_float2_to_fp4x2(make_float2(a, b), __NV_E2M1, cudaRoundNearest);
  const __half2_raw h = __nv_cvt_fp4x2_to_halfraw2(c, __NV_E2M1);
  const float2 q = __half22float2(*reinterpret_cast<const __half2*>(&h));
  *qa = q.x;
  *qb = q.y;
  return static_cast<uint32_t>(c);
}

// Eight threads (consecutive lanes) share one 32-element block, four consecutive values each: the 8-term split,
// for NB independent blocks at once (their dependency chains interleave).  `store(nb, t, bytes, se)` receives
// term t's two bytes of codes (values 0,1 and 2,3 of this thread) and the block exponent.  All 32 lanes must call
// it together.  (With NB > 1 the chains overlap little: the exchanges and the stores keep their program order.)
template <int NB, typename Store>
MOE_DEVINL void split_terms(float (&r)[NB][4], Store store) {
#pragma unroll 1
  for (int t = 0; t < kTerms; ++t) {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      float amax = fmaxf(fmaxf(fabsf(r[nb][0]), fabsf(r[nb][1])), fmaxf(fabsf(r[nb][2]), fabsf(r[nb][3])));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
      const int se = (amax > 0.0f) ? term_exp(amax) : 0;
      const float inv = pow2f(-se), sc = pow2f(se);
      float q0, q1, q2, q3;
      const uint32_t bytes =
          e2m1_pair(r[nb][0] * inv, r[nb][1] * inv, &q0, &q1) | (e2m1_pair(r[nb][2] * inv, r[nb][3] * inv, &q2, &q3) << 8);
      r[nb][0] = fmaf(-q0, sc, r[nb][0]);
      r[nb][1] = fmaf(-q1, sc, r[nb][1]);
      r[nb][2] = fmaf(-q2, sc, r[nb][2]);
      r[nb][3] = fmaf(-q3, sc, r[nb][3]);
      store(nb, t, bytes, se);
    }
  }
}

}  // namespace moe
