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
// Returns through lane j (< k) the j-th selected expert and its logit: experts in the order (logit descending by
// IEEE comparison, so -0 ties with +0; expert id ascending among equals).
// Up to 256 experts: a lane's eight logits stay in registers as integer keys that order like the floats (-0 counted
// as +0), so a round is a register max, two warp reductions and a few selects.
MOE_DEVINL void warp_topk_256(const float* row, int E, int k, int lane, int* my_id, float* my_v) {
  unsigned key[8];
  unsigned valid = 0u;  // bit u: element lane + 32*u exists and is not selected yet
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int idx = u * 32 + lane;
    const float v = idx < E ? row[idx] : 0.0f;
    const unsigned b = __float_as_uint(v == 0.0f ? 0.0f : v);
    key[u] = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    valid |= (idx < E ? 1u : 0u) << u;
  }
  *my_id = 0;
  *my_v = 0.0f;
  for (int j = 0; j < k; ++j) {
    unsigned best = 0u;
    bool any = false;
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if ((valid >> u) & 1u) {
        best = any ? max(best, key[u]) : key[u];
        any = true;
      }
    const unsigned top = __reduce_max_sync(0xffffffffu, any ? best : 0u);
    unsigned cand = 0xffffffffu;  // lowest id in this lane that holds the top key
#pragma unroll
    for (int u = 7; u >= 0; --u)
      if (((valid >> u) & 1u) && key[u] == top) cand = static_cast<unsigned>(u * 32 + lane);
    const unsigned win = __reduce_min_sync(0xffffffffu, cand);
    if ((win & 31u) == static_cast<unsigned>(lane)) valid &= ~(1u << (win >> 5));
    if (lane == j) {
      *my_id = static_cast<int>(win);
      *my_v = __uint_as_float((top & 0x80000000u) ? (top & 0x7fffffffu) : ~top);
    }
  }
}

MOE_DEVINL void warp_topk(const float* row, int E, int k, int lane, int* my_id, float* my_v) {
  if (E <= 256) {
    warp_topk_256(row, E, k, lane, my_id, my_v);
    return;
  }
  unsigned taken = 0u;  // bit i: element lane + 32*i already selected
  *my_id = 0;
  *my_v = 0.0f;
  for (int j = 0; j < k; ++j) {
    // this lane's best remaining element; strict '>': the lowest id among this lane's equal values stays
    float bv = 0.0f;
    int bi = -1;
    for (int i0 = 0; i0 * 32 < E; i0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = (i0 + u) * 32 + lane;
        v[u] = idx < E ? row[idx] : 0.0f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = (i0 + u) * 32 + lane;
        if (idx < E && !((taken >> (i0 + u)) & 1u) && (bi < 0 || v[u] > bv)) {
          bv = v[u];
          bi = idx;
        }
      }
    }
    // the warp's best: the largest value (as an integer key that orders floats, -0 counted as +0), then the lowest
    // id among the lanes that hold it; a lane with nothing left sends the lowest key and no id
    unsigned key = 0u;
    if (bi >= 0) {
      const unsigned u = __float_as_uint(bv == 0.0f ? 0.0f : bv);
      key = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    const unsigned best_key = __reduce_max_sync(0xffffffffu, key);
    const unsigned win = __reduce_min_sync(0xffffffffu, (bi >= 0 && key == best_key) ? static_cast<unsigned>(bi) : 0xffffffffu);
    const float win_v = __shfl_sync(0xffffffffu, bv, static_cast<int>(win & 31u));
    if ((win & 31u) == static_cast<unsigned>(lane)) taken |= 1u << (win >> 5);
    if (lane == j) {
      *my_id = static_cast<int>(win);
      *my_v = win_v;
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
