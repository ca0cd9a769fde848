// Expert FFN, weight-streaming variant: every touched expert's packed FP4 weights cross HBM once.
//
// Work item = (touched expert, tile of 16 weight rows) over the full K.  For the gate/up stage a tile
// is 8 gate rows (w1) plus the matching 8 up rows (w3), so silu(g)*u is local to a thread; for the down
// stage it is 16 consecutive rows of w2.  Rows of one expert matrix are contiguous in HBM, so a tile is
// one or two contiguous blocks that the producer warp brings into a shared-memory ring with bulk
// asynchronous copies (cp.async.bulk, completion on an mbarrier), packed: 4.25 bits per weight all the
// way to shared memory.  Sixteen consumer warps split K, expand E2M1 codes to bf16 in registers (the three
// magnitude bits dropped into the exponent/mantissa boundary of a bf16 give value * 2^-126 exactly; one
// packed multiply by 2^(scale byte - 1) restores value * 2^(scale byte - 127), also exactly), and feed
// m16n8k16 bf16 tensor-core MMAs whose n dimension holds up to 8 tokens of the expert.  Partial sums of
// the sixteen warps are added in a fixed order through shared memory, so the result is deterministic.
//
// K elements are assigned to MMA k slots in a permuted order (identically for weights and activations);
// only the summation order inside the dot product depends on it.
#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {

constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;  // + one producer warp
constexpr int kMaxScPerWarp = 2;                     // 128-element K groups a warp keeps activations for
constexpr int kSection = kConsumerWarps * kMaxScPerWarp * 128;  // K elements per register-resident pass

struct FfnArgs {
  const uint8_t* w;           // [E, R, K/2] packed codes
  const uint8_t* sc;          // [E, R, K/32] scale bytes
  const __nv_bfloat16* b;     // [S, K] activations (rows sorted by expert)
  const int* offsets;         // [E+1]
  __nv_bfloat16* act;         // stage 1 output [S, I]
  float* y;                   // stage 2 output [S, Hout]
  float* const* row_dst;      // or null; else output row p goes to row_dst[p] (see y_row)
  int* status;
  uint32_t k1, k2;         // 0x1040, 0x0104: multipliers of the E2M1 expansion, kept opaque to the compiler
  int E, K, R, I;             // R rows per expert (2I for stage 1, H for stage 2); I used by stage 1 only
  int n_stages;
};

MOE_DEVINL void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                 uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

}  // namespace

// STAGE1: tile = 8 gate rows + 8 up rows, epilogue = silu(g)*u -> bf16 act.
// !STAGE1: tile = 16 rows of w2, epilogue = fp32 store to y.
template <bool STAGE1>
__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(const FfnArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int K = a.K;
  const int code_half = 8 * (K / 2);   // bytes of 8 rows of codes
  const int scale_half = 8 * (K / 32); // bytes of 8 rows of scale bytes
  const int stage_bytes = 2 * (code_half + scale_half);
  const int n_stages = a.n_stages;

  unsigned char* ring = smem_raw;
  unsigned char* tail = smem_raw + static_cast<size_t>(n_stages) * stage_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail);         // [n_stages]
  uint64_t* empty_bar = full_bar + n_stages;                      // [n_stages]
  float* red = reinterpret_cast<float*>(empty_bar + n_stages);    // [2][kConsumerWarps][32][4]
  int* touched = reinterpret_cast<int*>(red + 2 * kConsumerWarps * 128);  // [E]
  int* s_misc = touched + a.E;                                    // [40]

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  // ---- list of touched experts (every CTA builds the same list) ----
  {
    const int per = (a.E + kThreads - 1) / kThreads;
    const int base = tid * per;
    int cnt = 0;
    for (int i = 0; i < per; ++i) {
      const int e = base + i;
      if (e < a.E && a.offsets[e + 1] > a.offsets[e]) ++cnt;
    }
    int wtot;
    const int ex = warp_excl_scan(cnt, lane, &wtot);
    if (lane == 0) s_misc[wid] = wtot;
    __syncthreads();
    if (wid == 0) {
      const int v = (lane < kThreads / 32) ? s_misc[lane] : 0;
      int tot;
      const int e2 = warp_excl_scan(v, lane, &tot);
      __syncwarp();
      s_misc[lane] = e2;
      if (lane == 0) s_misc[32] = tot;
    }
    __syncthreads();
    int pos = s_misc[wid] + ex;
    for (int i = 0; i < per; ++i) {
      const int e = base + i;
      if (e < a.E && a.offsets[e + 1] > a.offsets[e]) touched[pos++] = e;
    }
    if (tid == 0) {
      for (int s = 0; s < n_stages; ++s) {
        mbar_init(&full_bar[s], 1);
        mbar_init(&empty_bar[s], kConsumerWarps);
      }
      mbar_fence_init();
    }
    __syncthreads();
  }
  const int n_touched = s_misc[32];
  const int tiles_per_expert = a.R / 16;  // stage 1: I/8 (8 gate + 8 up rows each); stage 2: H/16
  const long long total_items = static_cast<long long>(n_touched) * tiles_per_expert;
  const long long per_cta = (total_items + gridDim.x - 1) / gridDim.x;
  const long long item_begin = static_cast<long long>(blockIdx.x) * per_cta;
  const long long item_end = min(item_begin + per_cta, total_items);

  const size_t w_expert = static_cast<size_t>(a.R) * (K / 2);
  const size_t s_expert = static_cast<size_t>(a.R) * (K / 32);

  if (wid == kConsumerWarps) {
    // ================= producer warp: one lane streams tiles into the ring =================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (long long it = item_begin; it < item_end; ++it) {
        const int e = touched[it / tiles_per_expert];
        const int tile = static_cast<int>(it % tiles_per_expert);
        mbar_wait(&empty_bar[stage], phase ^ 1u, a.status);
        unsigned char* dst = ring + static_cast<size_t>(stage) * stage_bytes;
        mbar_expect_tx(&full_bar[stage], static_cast<uint32_t>(stage_bytes));
        const uint8_t* wbase = a.w + e * w_expert;
        const uint8_t* sbase = a.sc + e * s_expert;
        if (STAGE1) {
          const int i0 = tile * 8;
          bulk_g2s(dst, wbase + static_cast<size_t>(i0) * (K / 2), code_half, &full_bar[stage]);
          bulk_g2s(dst + code_half, wbase + static_cast<size_t>(a.I + i0) * (K / 2), code_half, &full_bar[stage]);
          bulk_g2s(dst + 2 * code_half, sbase + static_cast<size_t>(i0) * (K / 32), scale_half, &full_bar[stage]);
          bulk_g2s(dst + 2 * code_half + scale_half, sbase + static_cast<size_t>(a.I + i0) * (K / 32), scale_half,
                   &full_bar[stage]);
        } else {
          const int r0 = tile * 16;
          bulk_g2s(dst, wbase + static_cast<size_t>(r0) * (K / 2), 2 * code_half, &full_bar[stage]);
          bulk_g2s(dst + 2 * code_half, sbase + static_cast<size_t>(r0) * (K / 32), 2 * scale_half,
                   &full_bar[stage]);
        }
        if (++stage == n_stages) {
          stage = 0;
          phase ^= 1u;
        }
      }
    }
  } else {
    // ================= consumer warps =================
    const int g = lane >> 2, t = lane & 3;
    const int n_sc = K / 128;                                // 128-element groups along K
    const int n_sections = (K + kSection - 1) / kSection;    // register-resident passes over K
    uint32_t breg[kMaxScPerWarp][16];                        // activations of row (n-tile, g), this lane's K slots
    int cached_row = -1;                                     // sorted row whose activations breg holds (-2: zeros)
    int stage = 0;
    uint32_t phase = 0;
    int red_buf = 0;
    int item_no = 0;

    for (long long it = item_begin; it < item_end; ++it, ++item_no) {
      const int e = touched[it / tiles_per_expert];
      const int tile = static_cast<int>(it % tiles_per_expert);
      const int row_begin = a.offsets[e], row_end = a.offsets[e + 1];
      mbar_wait(&full_bar[stage], phase, a.status);
      const unsigned char* st = ring + static_cast<size_t>(stage) * stage_bytes;
      const unsigned char* codesA = st;
      const unsigned char* codesB = st + code_half;
      const unsigned char* scaleA = st + 2 * code_half;
      const unsigned char* scaleB = scaleA + scale_half;

      for (int row0 = row_begin; row0 < row_end; row0 += 8) {
        float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        float c2[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // second chain: consecutive MMAs do not wait on each other
        const int my_row = (row0 + g < row_end) ? row0 + g : -2;
        for (int sec = 0; sec < n_sections; ++sec) {
          // ---- activations of this lane's row for this K section ----
          if (n_sections > 1 || my_row != cached_row) {
#pragma unroll
            for (int j = 0; j < kMaxScPerWarp; ++j) {
              const int sc = sec * (kConsumerWarps * kMaxScPerWarp) + j * kConsumerWarps + wid;
              if (sc < n_sc && my_row >= 0) {
                const uint4* src =
                    reinterpret_cast<const uint4*>(a.b + static_cast<size_t>(my_row) * K + sc * 128 + t * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const uint4 v = __ldcg(src + q);  // 8 consecutive elements
                  breg[j][4 * q + 0] = __byte_perm(v.x, v.z, 0x5410);  // elements (0,4)
                  breg[j][4 * q + 1] = __byte_perm(v.x, v.z, 0x7632);  // elements (1,5)
                  breg[j][4 * q + 2] = __byte_perm(v.y, v.w, 0x5410);  // elements (2,6)
                  breg[j][4 * q + 3] = __byte_perm(v.y, v.w, 0x7632);  // elements (3,7)
                }
              } else {
#pragma unroll
                for (int q = 0; q < 16; ++q) breg[j][q] = 0u;
              }
            }
            cached_row = my_row;
          }
          // ---- weights: dequantise and multiply ----
#pragma unroll
          for (int j = 0; j < kMaxScPerWarp; ++j) {
            const int sc = sec * (kConsumerWarps * kMaxScPerWarp) + j * kConsumerWarps + wid;
            if (sc < n_sc) {
              const uint4 wa = *reinterpret_cast<const uint4*>(codesA + g * (K / 2) + sc * 64 + t * 16);
              const uint4 wb = *reinterpret_cast<const uint4*>(codesB + g * (K / 2) + sc * 64 + t * 16);
              const uint32_t ma = scale_mult(scaleA[g * (K / 32) + sc * 4 + t]);
              const uint32_t mb = scale_mult(scaleB[g * (K / 32) + sc * 4 + t]);
              const uint32_t wav[4] = {wa.x, wa.y, wa.z, wa.w};
              const uint32_t wbv[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                uint32_t pa[4], pb[4];
                dequant8(wav[q], ma, a.k1, a.k2, pa);
                dequant8(wbv[q], mb, a.k1, a.k2, pb);
                mma_bf16_16x8x16(c, pa[0], pb[0], pa[1], pb[1], breg[j][4 * q + 0], breg[j][4 * q + 1]);
                mma_bf16_16x8x16(c2, pa[2], pb[2], pa[3], pb[3], breg[j][4 * q + 2], breg[j][4 * q + 3]);
              }
            }
          }
        }
        // ---- cross-warp reduction in fixed warp order, then the epilogue by one warp ----
        float* mine = red + ((red_buf * kConsumerWarps + wid) * 32 + lane) * 4;
        *reinterpret_cast<float4*>(mine) = make_float4(c[0] + c2[0], c[1] + c2[1], c[2] + c2[2], c[3] + c2[3]);
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
        if (wid == (item_no & (kConsumerWarps - 1))) {
          float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) {
            const float4 v = *reinterpret_cast<const float4*>(red + ((red_buf * kConsumerWarps + w) * 32 + lane) * 4);
            s.x += v.x;
            s.y += v.y;
            s.z += v.z;
            s.w += v.w;
          }
          // c0,c1: tile row g, tokens row0+2t, row0+2t+1; c2,c3: tile row g+8, same tokens
          const int r_a = row0 + 2 * t, r_b = r_a + 1;
          if (STAGE1) {
            const int i = tile * 8 + g;
            if (r_a < row_end) {
              const float v = (s.x / (1.0f + __expf(-s.x))) * s.z;
              a.act[static_cast<size_t>(r_a) * a.I + i] = __float2bfloat16_rn(v);
            }
            if (r_b < row_end) {
              const float v = (s.y / (1.0f + __expf(-s.y))) * s.w;
              a.act[static_cast<size_t>(r_b) * a.I + i] = __float2bfloat16_rn(v);
            }
          } else {
            const int n = tile * 16 + g;
            if (r_a < row_end) {
              float* ya = y_row(a.y, a.row_dst, static_cast<size_t>(r_a), a.R);
              ya[n] = s.x;
              ya[n + 8] = s.z;
            }
            if (r_b < row_end) {
              float* yb = y_row(a.y, a.row_dst, static_cast<size_t>(r_b), a.R);
              yb[n] = s.y;
              yb[n + 8] = s.w;
            }
          }
        }
        red_buf ^= 1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[stage]);
      if (++stage == n_stages) {
        stage = 0;
        phase ^= 1u;
      }
    }
  }
}

int launch_expert_ffn_stream(const __nv_bfloat16* x_perm, const int* offsets, const uint8_t* w13, const uint8_t* s13,
                      const uint8_t* w2, const uint8_t* s2, const moe_shape_t& sh, __nv_bfloat16* act, float* y_perm,
                      int* status_word, cudaStream_t st, float* const* row_dst) {
  constexpr int kSmemBudget = 200 * 1024;
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [] {
        return cudaFuncSetAttribute(ffn_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 24 * 1024) ==
                   cudaSuccess &&
               cudaFuncSetAttribute(ffn_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 24 * 1024) ==
                   cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  const int grid = sm_count();
  auto run = [&](bool stage1) -> bool {
    FfnArgs a;
    a.offsets = offsets;
    a.act = act;
    a.y = y_perm;
    a.row_dst = row_dst;
    a.status = status_word;
  a.k1 = 0x1040u;
  a.k2 = 0x0104u;
    a.k1 = 0x1040u;
    a.k2 = 0x0104u;
    a.E = sh.E;
    a.I = sh.I;
    if (stage1) {
      a.w = w13;
      a.sc = s13;
      a.b = x_perm;
      a.K = sh.H;
      a.R = 2 * sh.I;
    } else {
      a.w = w2;
      a.sc = s2;
      a.b = act;
      a.K = sh.I;
      a.R = sh.H;
    }
    const int stage_bytes = 16 * (a.K / 2 + a.K / 32);
    int n_stages = kSmemBudget / stage_bytes;
    if (n_stages > 12) n_stages = 12;
    if (n_stages < 2) return false;
    a.n_stages = n_stages;
    const size_t smem = static_cast<size_t>(n_stages) * stage_bytes + 2 * n_stages * 8 +
                        2 * kConsumerWarps * 128 * 4 + (static_cast<size_t>(sh.E) + 40) * 4;
    if (stage1)
      ffn_stream_kernel<true><<<grid, kThreads, smem, st>>>(a);
    else
      ffn_stream_kernel<false><<<grid, kThreads, smem, st>>>(a);
    return cudaGetLastError() == cudaSuccess;
  };
  if (!run(true)) return MOE_ERR_CUDA;
  if (!run(false)) return MOE_ERR_CUDA;
  note_kernel("ffn_stream_bulk_ring_mma16816", 2);
  return MOE_OK;
}

}  // namespace moe
