// Device routines of the router shared by moe_route's kernel and the one-launch decode kernel of moe_forward:
// the fixed fp32 exponential, the warp-wide top-k selection and the softmax over the selected logits.
#pragma once

#include "moe_common.cuh"

namespace moe {

// The fixed fp32 exponential of the routing softmax (sequence stated in the public header).  Every
// step is an explicitly rounded intrinsic so that the compiler cannot contract or reorder it.
MOE_DEVINL float exp_fixed(float d) {
  d = fmaxf(d, -80.0f);
  const float t = __fmul_rn(d, 0x1.715476p+0f);
  const float n = rintf(t);
  float r = __fmaf_rn(n, -0x1.62e4p-1f, d);
  r = __fmaf_rn(n, -0x1.7f7d1cp-20f, r);
  float p = 0x1.6c16c2p-10f;               // 1/720
  p = __fmaf_rn(p, r, 0x1.111112p-7f);     // 1/120
  p = __fmaf_rn(p, r, 0x1.555556p-5f);     // 1/24
  p = __fmaf_rn(p, r, 0x1.555556p-3f);     // 1/6
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  const int e = static_cast<int>(n);       // in [-116, 0]
  return __fmul_rn(p, __int_as_float((e + 127) << 23));
}

// One warp per token.  row = this warp's copy of the token's logits in shared memory.
// Returns through lane j (< k) the j-th selected expert and its logit.
MOE_DEVINL void warp_topk(const float* row, int E, int k, int lane, int* my_id, float* my_v) {
  unsigned taken = 0u;  // bit i: element lane + 32*i already selected
  *my_id = 0;
  *my_v = 0.0f;
  for (int j = 0; j < k; ++j) {
    float bv = 0.0f;
    int bi = -1;
    for (int i = 0; i * 32 + lane < E; ++i) {
      if (!((taken >> i) & 1u)) {
        const float v = row[i * 32 + lane];
        if (bi < 0 || v > bv) {  // strict '>': the lowest id among this lane's equal values stays
          bv = v;
          bi = i * 32 + lane;
        }
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, d);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, d);
      const bool take = (oi >= 0) && (bi < 0 || ov > bv || (ov == bv && oi < bi));
      if (take) {
        bv = ov;
        bi = oi;
      }
    }
    // lane 0's view is authoritative (identical on all lanes for finite logits)
    bi = __shfl_sync(0xffffffffu, bi, 0);
    bv = __shfl_sync(0xffffffffu, bv, 0);
    if (bi >= 0 && (bi & 31) == lane) taken |= 1u << (bi >> 5);
    if (lane == j) {
      *my_id = bi;
      *my_v = bv;
    }
  }
}

MOE_DEVINL float warp_softmax_selected(float my_v, int k, int lane) {
  const float m = __shfl_sync(0xffffffffu, my_v, 0);
  const float e = exp_fixed(__fsub_rn(my_v, m));
  float s = 0.0f;
  for (int j = 0; j < k; ++j) {
    const float ej = __shfl_sync(0xffffffffu, e, j);
    s = (j == 0) ? ej : __fadd_rn(s, ej);
  }
  return __fdiv_rn(e, s);
}

}  // namespace moe
