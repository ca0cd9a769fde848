// Expert FFN, tensor-core variant for prefill-sized batches: a persistent grouped GEMM on tcgen05.
//
// Roles inside the MMA: the M dimension (128 lanes of tensor memory) holds 128 weight rows, the N
// dimension holds up to 320 tokens of one expert (two accumulators, N <= 256 and N <= 64), so the
// padding of a ragged expert is at most 15 tokens and each packed weight is expanded once per pass.
// A work item is (expert, pass of <= 320 tokens, tile of 128 weight rows).  For the gate/up stage a tile
// is 64 gate rows (lanes 0..63) plus the matching 64 up rows (lanes 64..127).
//
// Warp roles (one CTA per SM, persistent):
//   warp 0      producer: TMA loads of the token tile (bf16, 128-byte swizzle) and of the packed codes
//   warp 1      allocates tensor memory, issues tcgen05.mma (one lane), commits to mbarriers
//   warps 2..9  expand E2M1 -> bf16 (exact, scaled by the E8M0 block scale) from the packed stage into the
//               swizzled K-major A stage the tensor core reads
//   warps 10..13 epilogue: tcgen05.ld the accumulators, SwiGLU + bf16 rounding (stage 1, gate and up meet
//               through shared memory) or the fp32 store (stage 2)
// Every mbarrier wait is bounded and reports through the status word.
#include <cuda.h>

#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {

constexpr int kTileM = 128;       // weight rows per tile
constexpr int kBlockK = 64;       // K per pipeline stage: one 128-byte row of bf16
constexpr int kMaxTok = 320;      // tokens per pass
constexpr int kTokBox = 64;       // token rows per TMA box
constexpr int kStages = 3;        // A/B ring depth
constexpr int kPackK = 256;       // K covered by one packed-code stage
constexpr int kPackStages = 2;
constexpr int kDequantWarps = 8;
constexpr int kEpilogueWarps = 4;
constexpr int kThreadsUmma = (2 + kDequantWarps + kEpilogueWarps) * 32;  // 448
constexpr int kFirstDequantWarp = 2;
constexpr int kFirstEpilogueWarp = 2 + kDequantWarps;  // 10: (warp % 4) = 2,3,0,1 covers the four lane quadrants
constexpr uint32_t kTmemCols = 512;

constexpr int kABytes = kTileM * kBlockK * 2;        // 16 KB
constexpr int kBBytes = kMaxTok * kBlockK * 2;       // 40 KB
constexpr int kPBytes = kTileM * (kPackK / 2);       // 16 KB
constexpr int kXchgBytes = 64 * 33 * 4;              // SwiGLU exchange: 64 up rows x 32 columns (+1 pad)

struct UmmaArgs {
  const uint8_t* sc;       // [E, R, K/32] scale bytes
  const int* offsets;      // [E+1]
  __nv_bfloat16* act;      // stage 1 output [S, I]
  float* y;                // stage 2 output [S, R]
  int* status;
  int E, K, R, I;          // R weight rows per expert (2I or H)
};

struct SmemMap {
  uint32_t a, b, p, xchg, bars, misc, prefix, total;
};
__host__ __device__ inline SmemMap smem_map(int E) {
  SmemMap m;
  uint32_t off = 0;
  m.a = off;
  off += kStages * kABytes;
  m.b = off;
  off += kStages * kBBytes;
  m.p = off;
  off += kPackStages * kPBytes;
  m.xchg = off;
  off += kXchgBytes;
  m.bars = off;
  off += 32 * 8;
  m.misc = off;
  off += 64;
  m.prefix = off;
  off += (static_cast<uint32_t>(E) + 2) * 4;
  m.total = off;
  return m;
}

// work id -> (expert, pass): prefix[e] = number of passes of experts < e
MOE_DEVINL int find_expert(const int* prefix, int E, int g) {
  int lo = 0, hi = E;  // invariant: prefix[lo] <= g < prefix[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= g) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace

template <bool STAGE1>
__global__ void __launch_bounds__(kThreadsUmma, 1)
ffn_umma_kernel(const __grid_constant__ CUtensorMap tmap_tok, const __grid_constant__ CUtensorMap tmap_w, const UmmaArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const SmemMap sm = smem_map(a.E);
  unsigned char* sA = smem + sm.a;
  unsigned char* sB = smem + sm.b;
  unsigned char* sP = smem + sm.p;
  float* sX = reinterpret_cast<float*>(smem + sm.xchg);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  uint64_t* full_a = bars;                      // [kStages] dequant warps -> MMA
  uint64_t* full_b = bars + kStages;            // [kStages] TMA -> MMA
  uint64_t* empty_ab = bars + 2 * kStages;      // [kStages] MMA done -> producer, dequant warps
  uint64_t* full_p = bars + 3 * kStages;        // [kPackStages] TMA -> dequant warps
  uint64_t* empty_p = full_p + kPackStages;     // [kPackStages] dequant warps -> producer
  uint64_t* acc_full = empty_p + kPackStages;   // MMA -> epilogue
  uint64_t* acc_empty = acc_full + 1;           // epilogue -> MMA
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sm.misc);
  int* prefix = reinterpret_cast<int*>(smem + sm.prefix);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int K = a.K;
  const int num_kb = K / kBlockK;
  const int tiles_per_expert = a.R / kTileM;

  // ---- setup: pass prefix over experts, barriers, tensor memory ----
  if (wid == 2) {
    // one warp builds the exclusive prefix of ceil(rows / kMaxTok) over experts
    int run = 0;
    for (int e0 = 0; e0 < a.E; e0 += 32) {
      const int e = e0 + lane;
      const int rows = (e < a.E) ? a.offsets[e + 1] - a.offsets[e] : 0;
      const int passes = (rows + kMaxTok - 1) / kMaxTok;
      int tot;
      const int ex = warp_excl_scan(passes, lane, &tot);
      if (e < a.E) prefix[e] = run + ex;
      run += tot;
    }
    if (lane == 0) prefix[a.E] = run;
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_a[s], kDequantWarps);
      mbar_init(&full_b[s], 1);
      mbar_init(&empty_ab[s], 1);
    }
    for (int s = 0; s < kPackStages; ++s) {
      mbar_init(&full_p[s], 1);
      mbar_init(&empty_p[s], kDequantWarps);
    }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, kEpilogueWarps);
    mbar_fence_init();
  }
  if (wid == 1) tmem_alloc(tmem_holder, kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  const int total_work = prefix[a.E] * tiles_per_expert;

  if (wid == 0) {
    // =========================== producer ===========================
    if (lane == 0) {
      int s = 0, ps = 0;
      uint32_t ph = 0, pph = 0;
      for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
        const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
        const int e = find_expert(prefix, a.E, g);
        const int pass = g - prefix[e];
        const int row0 = a.offsets[e] + pass * kMaxTok;
        const int ntok = min(kMaxTok, a.offsets[e + 1] - row0);
        const int nbox = (ntok + kTokBox - 1) / kTokBox;
        const int wrow_a = STAGE1 ? e * a.R + rt * 64 : e * a.R + rt * kTileM;
        const int wrow_b = STAGE1 ? e * a.R + a.I + rt * 64 : wrow_a + 64;
        for (int kb = 0; kb < num_kb; ++kb) {
          if ((kb & 3) == 0) {
            mbar_wait(&empty_p[ps], pph ^ 1u, a.status);
            mbar_expect_tx(&full_p[ps], kPBytes);
            unsigned char* dst = sP + ps * kPBytes;
            tma_load_2d(dst, &tmap_w, (kb >> 2) * (kPackK / 2), wrow_a, &full_p[ps]);
            tma_load_2d(dst + 64 * (kPackK / 2), &tmap_w, (kb >> 2) * (kPackK / 2), wrow_b, &full_p[ps]);
            if (++ps == kPackStages) { ps = 0; pph ^= 1u; }
          }
          mbar_wait(&empty_ab[s], ph ^ 1u, a.status);
          mbar_expect_tx(&full_b[s], static_cast<uint32_t>(nbox) * kTokBox * kBlockK * 2);
          for (int b = 0; b < nbox; ++b)
            tma_load_2d(sB + s * kBBytes + b * (kTokBox * kBlockK * 2), &tmap_tok, kb * kBlockK, row0 + b * kTokBox,
                        &full_b[s]);
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (wid == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0, acc_ph = 0;
      for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
        const int g = w / tiles_per_expert;
        const int e = find_expert(prefix, a.E, g);
        const int pass = g - prefix[e];
        const int row0 = a.offsets[e] + pass * kMaxTok;
        const int ntok = min(kMaxTok, a.offsets[e + 1] - row0);
        const int n16 = (ntok + 15) & ~15;
        const int n1 = min(n16, 256), n2 = n16 - n1;
        const uint32_t idesc1 = umma_idesc_bf16(kTileM, n1);
        const uint32_t idesc2 = umma_idesc_bf16(kTileM, n2 > 0 ? n2 : 16);
        mbar_wait(acc_empty, acc_ph ^ 1u, a.status);
        tc_fence_after_sync();
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(&full_a[s], ph, a.status);
          mbar_wait(&full_b[s], ph, a.status);
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(sA + s * kABytes);
          const uint32_t b_addr = smem_u32(sB + s * kBBytes);
#pragma unroll
          for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
            const uint64_t adesc = umma_desc_k_sw128(a_addr + k4 * 32);
            const uint32_t acc = (kb | k4) != 0 ? 1u : 0u;
            umma_bf16(tmem_base, adesc, umma_desc_k_sw128(b_addr + k4 * 32), idesc1, acc);
            if (n2 > 0) umma_bf16(tmem_base + 256, adesc, umma_desc_k_sw128(b_addr + 256 * 128 + k4 * 32), idesc2, acc);
          }
          umma_commit(&empty_ab[s]);
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        umma_commit(acc_full);
        acc_ph ^= 1u;
      }
    }
  } else if (wid < kFirstEpilogueWarp) {
    // =========================== E2M1 -> bf16 expansion ===========================
    const int dt = tid - kFirstDequantWarp * 32;  // 0..255
    const int row = dt >> 1, half = dt & 1;       // tile row, which 32 elements of the 64-wide K block
    int s = 0, ps = 0;
    uint32_t ph = 0, pph = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
      const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
      const int e = find_expert(prefix, a.E, g);
      const int grow = STAGE1 ? e * a.R + (row < 64 ? rt * 64 + row : a.I + rt * 64 + (row - 64)) : e * a.R + rt * kTileM + row;
      const uint8_t* srow = a.sc + static_cast<size_t>(grow) * (K / 32);
      for (int kb = 0; kb < num_kb; ++kb) {
        if ((kb & 3) == 0) mbar_wait(&full_p[ps], pph, a.status);
        const uint32_t scale_byte = __ldg(srow + kb * 2 + half);
        const uint4 codes = *reinterpret_cast<const uint4*>(sP + ps * kPBytes + row * (kPackK / 2) + (kb & 3) * 32 + half * 16);
        const uint32_t m = scale_mult(scale_byte);
        const uint32_t wv[4] = {codes.x, codes.y, codes.z, codes.w};
        uint4 out[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t p[4];
          dequant8(wv[q], m, p);
          // (0,4),(1,5),(2,6),(3,7) -> natural order (0,1),(2,3),(4,5),(6,7)
          out[q].x = __byte_perm(p[0], p[1], 0x5410);
          out[q].y = __byte_perm(p[2], p[3], 0x5410);
          out[q].z = __byte_perm(p[0], p[1], 0x7632);
          out[q].w = __byte_perm(p[2], p[3], 0x7632);
        }
        mbar_wait(&empty_ab[s], ph ^ 1u, a.status);
        unsigned char* arow = sA + s * kABytes + row * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int chunk = half * 4 + q;  // 16-byte chunk of the 128-byte row
          *reinterpret_cast<uint4*>(arow + ((chunk ^ (row & 7)) << 4)) = out[q];
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&full_a[s]);
          if ((kb & 3) == 3) mbar_arrive(&empty_p[ps]);
        }
        if ((kb & 3) == 3) {
          if (++ps == kPackStages) { ps = 0; pph ^= 1u; }
        }
        if (++s == kStages) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // =========================== epilogue ===========================
    const int q = wid & 3;  // tensor-memory lane quadrant this warp may read
    const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
    uint32_t acc_ph = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
      const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
      const int e = find_expert(prefix, a.E, g);
      const int pass = g - prefix[e];
      const int row0 = a.offsets[e] + pass * kMaxTok;
      const int ntok = min(kMaxTok, a.offsets[e + 1] - row0);
      mbar_wait(acc_full, acc_ph, a.status);
      tc_fence_after_sync();
      for (int c0 = 0; c0 < ntok; c0 += 32) {
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + lane_base + static_cast<uint32_t>(c0), v);
        tmem_ld_wait();
        if (STAGE1) {
          // lanes 0..63 hold gate rows, lanes 64..127 the matching up rows: up goes through shared memory
          if (q >= 2) {
#pragma unroll
            for (int j = 0; j < 32; ++j) sX[((q - 2) * 32 + lane) * 33 + j] = __uint_as_float(v[j]);
          }
          asm volatile("bar.sync 2, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
          if (q < 2) {
            const int i = rt * 64 + q * 32 + lane;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < ntok) {
                const float gv = __uint_as_float(v[j]);
                const float uv = sX[(q * 32 + lane) * 33 + j];
                const float r = (gv / (1.0f + __expf(-gv))) * uv;
                a.act[static_cast<size_t>(row0 + c0 + j) * a.I + i] = __float2bfloat16_rn(r);
              }
            }
          }
          asm volatile("bar.sync 2, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
        } else {
          const int n = rt * kTileM + q * 32 + lane;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c0 + j < ntok) a.y[static_cast<size_t>(row0 + c0 + j) * a.R + n] = __uint_as_float(v[j]);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty);
      acc_ph ^= 1u;
    }
  }

  // ---- teardown ----
  tc_fence_before_sync();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- host side ---------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool make_map_2d(CUtensorMap* m, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner, uint64_t rows,
                 uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * static_cast<uint64_t>(elem_bytes)};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool umma_shape_ok(const moe_shape_t& sh) {
  return sh.H % kPackK == 0 && sh.I % kPackK == 0 && static_cast<long long>(sh.T) * sh.k >= 1024 &&
         smem_map(sh.E).total + 1024 <= 227 * 1024;
}

int launch_expert_ffn_umma(const __nv_bfloat16* x_perm, const int* offsets, const uint8_t* w13, const uint8_t* s13,
                           const uint8_t* w2, const uint8_t* s2, const moe_shape_t& sh, __nv_bfloat16* act, float* y_perm,
                           int* status_word, cudaStream_t st) {
  const size_t smem = smem_map(sh.E).total + 1024;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(ffn_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(ffn_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return MOE_ERR_CUDA;
    attr_done = true;
  }
  const uint64_t S = static_cast<uint64_t>(sh.T) * sh.k;
  CUtensorMap tm_x, tm_act, tm_w13, tm_w2;
  if (!make_map_2d(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x_perm, sh.H, S, kBlockK, kTokBox, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map_2d(&tm_act, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, act, sh.I, S, kBlockK, kTokBox, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map_2d(&tm_w13, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w13, sh.H / 2, static_cast<uint64_t>(sh.E) * 2 * sh.I,
                   kPackK / 2, 64, CU_TENSOR_MAP_SWIZZLE_NONE) ||
      !make_map_2d(&tm_w2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w2, sh.I / 2, static_cast<uint64_t>(sh.E) * sh.H, kPackK / 2, 64,
                   CU_TENSOR_MAP_SWIZZLE_NONE))
    return MOE_ERR_CUDA;
  const int grid = sm_count();
  UmmaArgs a;
  a.offsets = offsets;
  a.act = act;
  a.y = y_perm;
  a.status = status_word;
  a.E = sh.E;
  a.I = sh.I;
  a.sc = s13;
  a.K = sh.H;
  a.R = 2 * sh.I;
  ffn_umma_kernel<true><<<grid, kThreadsUmma, smem, st>>>(tm_x, tm_w13, a);
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  a.sc = s2;
  a.K = sh.I;
  a.R = sh.H;
  ffn_umma_kernel<false><<<grid, kThreadsUmma, smem, st>>>(tm_act, tm_w2, a);
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  note_kernel("ffn_umma_tcgen05_grouped", 2);
  return MOE_OK;
}

}  // namespace moe
